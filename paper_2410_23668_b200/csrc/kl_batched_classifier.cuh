// Classifier for a batch of sequences on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
//   logits[b, v] = sum_k W_lm[v, k] * xn[b, k],   xn[b] = rmsnorm(x[b]; g_f),   b < B <= 32
//
// At batch 32 this projection is a dense contraction (the operation-intensity table of the paper, Table 1: ~20 FLOP/B
// at B = 32): W_lm is streamed ONCE for all sequences.  Tiling: a CTA owns row tiles of 128 vocabulary rows
// (M = 128); the normalised inputs enter as the N operand, split into bf16 hi and lo halves that sit in columns
// 0..31 and 32..63 of ONE N = 64 operand, so a single MMA per 16 columns of K produces W.x_hi and W.x_lo side by
// side and the epilogue adds them (fp32-accurate inputs on a bf16 tensor pipe).  Per 64 columns of K one stage of the
// shared-memory ring holds a [128 x 64] tile of W_lm (16 KB) and the [64 x 64] tile of the inputs (8 KB), both
// written by TMA with the 128-byte swizzle that the MMA's shared-memory descriptors expect.
//
// Roles (192 threads): warp 0 lane 0 issues the TMA loads; warp 1 allocates TMEM and its lane 0 issues the MMAs
// (tcgen05.mma, cta_group::1, kind::f16, M 128 x N 64 x K 16) and the commits; warps 2..5 are the epilogue: each
// reads its 32 TMEM lanes (tcgen05.ld 32x32b) and stores logits.  Two accumulator buffers (2 x 64 TMEM columns) let
// the epilogue of one tile overlap the MMAs of the next.  Every mbarrier wait is bounded; on a time-out the kernel
// sets the status word, stops issuing, and every role falls through to the common exit (TMEM is freed there).
#pragma once

namespace kl {

constexpr int BC_THREADS = 192;
constexpr int BC_STAGES = 6;
constexpr int BC_TILE_M = 128;
constexpr int BC_TILE_N = 64;   // 32 sequences x (hi, lo)
constexpr int BC_TILE_K = 64;   // bf16 columns per stage = one 128-byte swizzle row
constexpr int BC_A_BYTES = BC_TILE_M * BC_TILE_K * 2;
constexpr int BC_B_BYTES = BC_TILE_N * BC_TILE_K * 2;
constexpr int BC_STAGE_BYTES = BC_A_BYTES + BC_B_BYTES;
constexpr int BC_TMEM_COLS = 128;   // two accumulator buffers of 64 fp32 columns
constexpr size_t BC_SMEM_BYTES = (size_t)BC_STAGES * BC_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

struct BcParams {
    CUtensorMap map_w;     // W_lm as [V rows, H cols] bf16, box 64 x 128, 128-byte swizzle
    CUtensorMap map_x;     // inputs as [64 rows, H cols] bf16 (rows 0..31 hi halves, 32..63 lo halves), box 64 x 64
    float* logits;         // [B, V]
    uint32_t V, H, B;
    int32_t* status;
    uint64_t wait_ns;
};

// ---- PTX wrappers (tcgen05 / TMEM)

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

__device__ __forceinline__ bool bc_wait(uint32_t bar, uint32_t parity, const BcParams& p, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = globaltimer_ns();
    uint32_t it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 63u) == 0) {
            if (*abort_flag) return false;
            if (globaltimer_ns() - t0 > p.wait_ns) {
                atomicCAS(p.status, 0, ERR_SYNC_TIMEOUT);
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}

// Normalised inputs as the N operand: xb[b][k] = hi half, xb[32 + b][k] = lo half of x[b][k] * rsqrt(mean x^2 + eps) * g[k];
// rows of sequences >= B are zero.  One block per sequence slot (32 blocks).
__global__ void __launch_bounds__(256) kl_bc_prepare_kernel(const float* hidden, const __nv_bfloat16* gain, __nv_bfloat16* xb,
                                                            uint32_t H, uint32_t B, float eps) {
    const uint32_t b = blockIdx.x, tid = threadIdx.x;
    __shared__ float red[8];
    __nv_bfloat16* hi = xb + (size_t)b * H;
    __nv_bfloat16* lo = xb + (size_t)(32 + b) * H;
    if (b >= B) {
        for (uint32_t k = tid; k < H; k += blockDim.x) hi[k] = lo[k] = __float2bfloat16_rn(0.f);
        return;
    }
    const float* x = hidden + (size_t)b * H;
    float ss = 0.f;
    for (uint32_t k = tid; k < H; k += blockDim.x) ss += x[k] * x[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)H + eps);
    for (uint32_t k = tid; k < H; k += blockDim.x) {
        const float v = x[k] * __bfloat162float(gain[k]) * inv;
        const __nv_bfloat16 h16 = __float2bfloat16_rn(v);
        hi[k] = h16;
        lo[k] = __float2bfloat16_rn(v - __bfloat162float(h16));
    }
}

__global__ void __launch_bounds__(BC_THREADS, 1) kl_bc_kernel(const __grid_constant__ BcParams p) {
    extern __shared__ uint8_t bc_smem_raw[];
    // tiles on 1024-byte boundaries (the swizzle pattern repeats every 1024 bytes)
    const uint32_t raw = smem_u32(bc_smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t* misc = bc_smem_raw + (tiles - raw) + (size_t)BC_STAGES * BC_STAGE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(misc);            // [BC_STAGES] tile pair landed
    uint64_t* empty = full + BC_STAGES;                             // [BC_STAGES] MMAs that read the stage are done
    uint64_t* acc_full = empty + BC_STAGES;                         // [2] accumulator buffer complete
    uint64_t* acc_empty = acc_full + 2;                             // [2] epilogue has read the buffer
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_s + 1);

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < BC_STAGES; ++i) {
            mbar_init(smem_u32(&full[i]), 1);
            mbar_init(smem_u32(&empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&acc_full[i]), 1);
            mbar_init(smem_u32(&acc_empty[i]), 4);   // one arrival per epilogue warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_base_s), BC_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_s;

    const uint32_t ntiles = (p.V + BC_TILE_M - 1) / BC_TILE_M;
    const uint32_t nkb = p.H / BC_TILE_K;
    const bool skip = *p.status != 0;   // an earlier kernel of this step flagged an error: the step is a no-op

    if (!skip && warp == 0 && lane == 0) {
        // ---- producer: TMA loads of the W tile and the input tile of every (row tile, K block)
        const uint64_t pol = l2_policy_evict_first();
        uint32_t stage = 0, use = 0;
        for (uint32_t t = blockIdx.x; t < ntiles && !*abort_flag; t += gridDim.x) {
            for (uint32_t kb = 0; kb < nkb; ++kb) {
                if (use > 0 && !bc_wait(smem_u32(&empty[stage]), (use - 1u) & 1u, p, abort_flag)) break;
                const uint32_t bar = smem_u32(&full[stage]);
                const uint32_t dst = tiles + stage * BC_STAGE_BYTES;
                mbar_arrive_expect_tx(bar, (uint32_t)BC_STAGE_BYTES);
                tma_tensor_2d_g2s(dst, &p.map_w, (int32_t)(kb * BC_TILE_K), (int32_t)(t * BC_TILE_M), bar, pol);
                tma_tensor_2d_g2s(dst + BC_A_BYTES, &p.map_x, (int32_t)(kb * BC_TILE_K), 0, bar, pol);
                if (++stage == BC_STAGES) {
                    stage = 0;
                    ++use;
                }
            }
        }
        if (*abort_flag) {
            // no copy may still be writing this CTA's shared memory when it exits: wait (bounded) for the last copy
            // armed on every stage
            const uint64_t t0 = globaltimer_ns();
            for (uint32_t sidx = 0; sidx < (uint32_t)BC_STAGES; ++sidx) {
                const uint32_t cnt = use + (sidx < stage ? 1u : 0u);
                if (cnt == 0) continue;
                while (!mbar_try_wait(smem_u32(&full[sidx]), (cnt - 1u) & 1u))
                    if (globaltimer_ns() - t0 > p.wait_ns) break;
            }
        }
    } else if (!skip && warp == 1 && lane == 0) {
        // ---- MMA issuer
        const uint32_t idesc = umma_idesc_bf16(BC_TILE_M, BC_TILE_N);
        uint32_t stage = 0, use = 0, it = 0;
        for (uint32_t t = blockIdx.x; t < ntiles && !*abort_flag; t += gridDim.x, ++it) {
            const uint32_t buf = it & 1u, buse = it >> 1;
            if (buse > 0 && !bc_wait(smem_u32(&acc_empty[buf]), (buse - 1u) & 1u, p, abort_flag)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + buf * BC_TILE_N;
            for (uint32_t kb = 0; kb < nkb; ++kb) {
                if (!bc_wait(smem_u32(&full[stage]), use & 1u, p, abort_flag)) break;
                tc_fence_after();
                const uint32_t a_addr = tiles + stage * BC_STAGE_BYTES;
                const uint64_t a_desc = umma_desc_sw128(a_addr), b_desc = umma_desc_sw128(a_addr + BC_A_BYTES);
#pragma unroll
                for (uint32_t k = 0; k < BC_TILE_K / 16; ++k)   // 16 bf16 = 32 bytes further along the swizzled row
                    umma_f16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0u);
                umma_commit(smem_u32(&empty[stage]));   // the stage may be refilled when these MMAs are done
                if (++stage == BC_STAGES) {
                    stage = 0;
                    ++use;
                }
            }
            umma_commit(smem_u32(&acc_full[buf]));
        }
    } else if (!skip && warp >= 2) {
        // ---- epilogue: warp w reads TMEM lanes 32 * (w % 4) .. + 31 = rows of the tile
        const uint32_t quarter = warp & 3u;
        uint32_t it = 0;
        for (uint32_t t = blockIdx.x; t < ntiles; t += gridDim.x, ++it) {
            const uint32_t buf = it & 1u, buse = it >> 1;
            if (!bc_wait(smem_u32(&acc_full[buf]), buse & 1u, p, abort_flag)) break;
            tc_fence_after();
            uint32_t hi[32], lo[32];
            const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + buf * BC_TILE_N;
            tmem_ld32(taddr, hi);
            tmem_ld32(taddr + 32u, lo);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
            const uint32_t row = t * BC_TILE_M + quarter * 32u + lane;
            if (row < p.V) {
#pragma unroll
                for (uint32_t b = 0; b < 32; ++b)
                    if (b < p.B) p.logits[(size_t)b * p.V + row] = __uint_as_float(hi[b]) + __uint_as_float(lo[b]);
            }
        }
    }
    // ---- common exit: nobody may still be using TMEM when it is freed
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BC_TMEM_COLS);
    }
}

}  // namespace kl
