// Prompt processing on the 5th-generation tensor cores.
//
// The decode path streams every weight once per <= 16 rows; for a prompt of hundreds of rows that is the wrong
// trade.  Here a block of up to PF_ROWS prompt rows goes through a layer as real GEMMs: C[rows, N] = A[rows, K] W[N, K]^T
// with 128 x 128 output tiles, operands brought into shared memory by TMA tensor copies (64-column boxes, 128-byte
// swizzle), tcgen05.mma issued by one thread with the accumulators in tensor memory, and an epilogue that reads
// them back with tcgen05.ld.  The activations keep fp32 accuracy the same way as in the decode path: every value
// is split into two bf16 planes, x = hi + lo, and both planes are multiplied with the bf16 weights into the same
// fp32 accumulator.  The tensor core's fp32 accumulation rounds toward zero, which biases long chains; every k block
// of 64 therefore gets a fresh accumulator (four rotate through the 512 tensor-memory columns) that the epilogue
// warps add to fp32 registers while the next blocks are being multiplied.
//
// Around the GEMMs sit small elementwise kernels (embedding gather, RMSNorm + split into planes, SwiGLU + split,
// RoPE + KV append) and the tensor-core attention of the decode path run over (row block, head) items.
#pragma once

#include <cuda.h>

#include "kg_device.cuh"

namespace kg {

constexpr int PF_ROWS = 512;            // prompt rows per pass through the layers
constexpr int GM_BM = 128, GM_BN = 128, GM_BK = 64;
constexpr int GM_STAGES = 4;
constexpr int GM_TILE_BYTES = GM_BM * GM_BK * 2;                       // one 128 x 64 bf16 tile: 16 KB
constexpr int GM_STAGE_BYTES = 3 * GM_TILE_BYTES;                      // A hi, A lo, W
constexpr int GM_SMEM = GM_STAGES * GM_STAGE_BYTES + 1024 + 256;       // + alignment slack + barriers
constexpr int GM_THREADS = 320;                                        // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr int GM_EPI_WARPS = 8;                                        // two per tensor-memory lane quadrant, 64 columns each
constexpr int GM_ACC = 4;                                              // rotating accumulators of 128 columns (= stages)
constexpr unsigned long long GM_WAIT_CLK = 4000000000ull;              // ~2 s: a wait that runs this long gives up

struct GemmArgs {
    float* C; int ldc;                  // [rows, N] fp32
    float* C2;                          // grid.z == 2: the output of the second weight matrix (same shape, same A)
    const float* resid; int ldr;        // optional: C = resid + rowscale * A W^T
    const float* rowscale;              // optional: one factor per row (1/rms of the row the planes were made from)
    int rows;                           // valid rows (the planes hold a multiple of 128, zero beyond)
    int N, K;                           // multiples of 128 and 64
    int* err;                           // set to 1 when a bounded wait expired
};

// ---- TMA tile copy, tensor memory and tcgen05 MMA ----------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* tmap, int x, int y, uint32_t bar_smem) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst_smem), "l"(tmap), "r"(x), "r"(y), "r"(bar_smem) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle (rows of 128 bytes, groups of 8 rows 1024 bytes apart).
// bits [0,14) address >> 4, [32,46) group stride >> 4, [46,48) version 1, [61,64) layout 2 = 128-byte swizzle.
// Stepping 16 k-elements inside the 64-element atom adds 32 bytes (2 units) to the address field.
constexpr uint32_t UMMA_DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | (1u << 16); }
// Instruction descriptor: fp32 accumulate (bit 4), bf16 A and B (bits 7, 10), both K-major, N >> 3 at bit 17, M >> 4 at bit 24.
__device__ __forceinline__ uint32_t umma_idesc_128(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}
// D[128 x N] (+)= A[128 x 16] B[N x 16]^T, issued by one thread
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                 ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(UMMA_DESC_HI), "r"(idesc), "r"(accumulate));
}
// the mbarrier receives one arrival when every MMA this thread has issued so far has completed
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive accumulator columns of this thread's tensor-memory lane (lane = 32 * (warp % 4) + lane id)
// (asynchronous: tmem_ld_wait() before the values are used)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// bounded wait on an mbarrier phase; on expiry the error word is set and false returned
__device__ __forceinline__ bool gm_wait(unsigned long long* bar, unsigned parity, int* err) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (((++spins) & 255u) == 0u) {
            if (*(volatile int*)err) return false;
            if ((unsigned long long)(clock64() - t0) > GM_WAIT_CLK) { *(volatile int*)err = 1; return false; }
        }
    }
    return true;
}

// ---- the GEMM ------------------------------------------------------------------------------------------------------
// grid = (N / 128, row tiles, 1 or 2 weight matrices that share A); one 128 x 128 tile of C per CTA.  k block kb uses shared-memory stage kb mod 4 and
// tensor-memory accumulator kb mod 4: its eight MMAs (four k16-steps, hi and lo plane) start a fresh accumulator, one
// tcgen05.commit tells the producer that the stage is free and the epilogue warps that the accumulator is complete,
// and the epilogue warps add it to their fp32 registers (round to nearest) and hand the accumulator back.  No sum
// therefore passes through more than eight of the tensor core's truncating accumulations.
__global__ void __launch_bounds__(GM_THREADS, 1) pf_gemm_kernel(const __grid_constant__ CUtensorMap tm_hi, const __grid_constant__ CUtensorMap tm_lo,
                                                                const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_w2,
                                                                const GemmArgs g) {
    extern __shared__ __align__(128) char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    char* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);              // swizzled tiles sit on 1024-byte boundaries
    unsigned long long* full = reinterpret_cast<unsigned long long*>(smem + GM_STAGES * GM_STAGE_BYTES);   // TMA -> MMA: stage filled
    unsigned long long* mma_done = full + GM_STAGES;      // MMA -> TMA, epilogue: the k block's MMAs have completed
    unsigned long long* acc_free = mma_done + GM_STAGES;  // epilogue -> MMA: the accumulator has been read (one arrival per warp)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_free + GM_ACC);
    static_assert(GM_STAGES == GM_ACC, "a k block's stage and accumulator share one index and one completion barrier");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * GM_BN, m0 = blockIdx.y * GM_BM;
    const int nkb = g.K / GM_BK;
    const CUtensorMap* tm_wz = blockIdx.z ? &tm_w2 : &tm_w;
    float* Cz = blockIdx.z ? g.C2 : g.C;
    if (threadIdx.x == 0) {
        for (int i = 0; i < GM_STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&mma_done[i], 1); mbar_init(&acc_free[i], GM_EPI_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ---- TMA producer: A hi, A lo and W boxes of one k block per stage
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % GM_STAGES;
            if (!gm_wait(&mma_done[s], ((unsigned)(kb / GM_STAGES) & 1u) ^ 1u, g.err)) break;
            const uint32_t dst = smem_u32(smem + s * GM_STAGE_BYTES), bar = smem_u32(&full[s]);
            mbar_arrive_expect_tx(&full[s], (unsigned)GM_STAGE_BYTES);
            tma_load_2d(dst, &tm_hi, kb * GM_BK, m0, bar);
            tma_load_2d(dst + GM_TILE_BYTES, &tm_lo, kb * GM_BK, m0, bar);
            tma_load_2d(dst + 2 * GM_TILE_BYTES, tm_wz, kb * GM_BK, n0, bar);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        const uint32_t idesc = umma_idesc_128(GM_BN);
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % GM_STAGES;
            const unsigned par = (unsigned)(kb / GM_STAGES) & 1u;
            if (!gm_wait(&acc_free[s], par ^ 1u, g.err)) break;
            if (!gm_wait(&full[s], par, g.err)) break;
            tc_fence_after();
            const uint32_t a_hi = umma_desc_lo(smem_u32(smem + s * GM_STAGE_BYTES));
            const uint32_t a_lo = umma_desc_lo(smem_u32(smem + s * GM_STAGE_BYTES + GM_TILE_BYTES));
            const uint32_t w = umma_desc_lo(smem_u32(smem + s * GM_STAGE_BYTES + 2 * GM_TILE_BYTES));
            const uint32_t d = tmem + (uint32_t)s * GM_BN;
#pragma unroll
            for (int k16 = 0; k16 < GM_BK / 16; ++k16) {
                umma_bf16(d, a_hi + 2u * k16, w + 2u * k16, idesc, k16 > 0 ? 1u : 0u);
                umma_bf16(d, a_lo + 2u * k16, w + 2u * k16, idesc, 1u);
            }
            umma_commit(&mma_done[s]);
        }
    } else if (warp >= 2) {
        // ---- epilogue: thread = one row of the tile (tensor-memory lane = 32 * (warp % 4) + lane id) and one half of its
        // columns (warps 2-5: columns 0-63, warps 6-9: 64-127); the 64 sums live in registers
        const int q = warp & 3;
        const int ch = ((warp - 2) >> 2) * (GM_BN / 2);
        const int row = m0 + q * 32 + lane;
        float acc[GM_BN / 2];
#pragma unroll
        for (int i = 0; i < GM_BN / 2; ++i) acc[i] = 0.f;
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int s = kb % GM_ACC;
            ok = gm_wait(&mma_done[s], (unsigned)(kb / GM_ACC) & 1u, g.err);
            if (!ok) break;
            tc_fence_after();
            uint32_t v0[32], v1[32];
            const uint32_t ta = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(s * GM_BN + ch);
            tmem_ld32(ta, v0);
            tmem_ld32(ta + 32u, v1);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) { acc[i] += __uint_as_float(v0[i]); acc[32 + i] += __uint_as_float(v1[i]); }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_free[s]);
        }
        if (ok && row < g.rows) {
            float* dst = Cz + (size_t)row * g.ldc + n0 + ch;
            if (g.rowscale) {
                const float rsc = g.rowscale[row];
#pragma unroll
                for (int i = 0; i < GM_BN / 2; ++i) acc[i] *= rsc;
            }
            if (g.resid) {
                const float* rs = g.resid + (size_t)row * g.ldr + n0 + ch;
#pragma unroll
                for (int i = 0; i < GM_BN / 2; i += 4) {
                    const float4 r4 = *reinterpret_cast<const float4*>(rs + i);
                    acc[i] += r4.x; acc[i + 1] += r4.y; acc[i + 2] += r4.z; acc[i + 3] += r4.w;
                }
            }
#pragma unroll
            for (int i = 0; i < GM_BN / 2; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// ---- elementwise kernels around the GEMMs ----------------------------------------------------------------------------
__device__ __forceinline__ void split_store(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    hi[i] = h;
    lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

// h[r] = E[token r]
template <typename WT>
__global__ void pf_embed_kernel(const int* toks, const WT* E, int V, int d, float* h) {
    const int r = blockIdx.x;
    int tok = toks[r];
    if ((unsigned)tok >= (unsigned)V) tok = 0;
    for (int e = threadIdx.x; e < d; e += blockDim.x) h[(size_t)r * d + e] = wt_to_float<WT>(E[(size_t)tok * d + e]);
}

// four consecutive values -> four bf16 of each plane (8-byte stores; i is a multiple of 4)
__device__ __forceinline__ void split_store4(__nv_bfloat16* hi, __nv_bfloat16* lo, size_t i, float4 v) {
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
    const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
    const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - f0.x, v.y - f0.y), l1 = __floats2bfloat162_rn(v.z - f1.x, v.w - f1.y);
    uint2 hv, lv;
    hv.x = *reinterpret_cast<const unsigned*>(&h0); hv.y = *reinterpret_cast<const unsigned*>(&h1);
    lv.x = *reinterpret_cast<const unsigned*>(&l0); lv.y = *reinterpret_cast<const unsigned*>(&l1);
    *reinterpret_cast<uint2*>(hi + i) = hv;
    *reinterpret_cast<uint2*>(lo + i) = lv;
}

// planes of x[r] * gain and rs[r] = 1 / rms(x[r]): the GEMM that reads the
// planes multiplies its rows by rs afterwards, in fp32, exactly as the decode path's linear operator does (values that
// are exact in bf16, such as embedding rows under a unit gain, then stay exact).  One CTA of PF_EW_THREADS threads per
// row; the row (K a multiple of 4, at most PF_EW_THREADS * 4 * PF_NORM_V values) is read once and kept in registers.
constexpr int PF_EW_THREADS = 256;
constexpr int PF_NORM_V = 8;                  // float4 per thread: rows of up to 8192 values
__global__ void __launch_bounds__(PF_EW_THREADS) pf_norm_split_kernel(const float* x, int ldx, int K, const float* gain, float eps,
                                                                      __nv_bfloat16* hi, __nv_bfloat16* lo, float* rs) {
    __shared__ float red[32];
    const int r = blockIdx.x;
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)r * ldx);
    const int n4 = K >> 2;
    float4 v[PF_NORM_V];
#pragma unroll
    for (int j = 0; j < PF_NORM_V; ++j) {
        const int i = threadIdx.x + j * PF_EW_THREADS;
        v[j] = i < n4 ? xr[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    {
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < PF_NORM_V; ++j) ss += (v[j].x * v[j].x + v[j].y * v[j].y) + (v[j].z * v[j].z + v[j].w * v[j].w);
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x < 32) {
            float t = threadIdx.x < (PF_EW_THREADS >> 5) ? red[threadIdx.x] : 0.f;
            t = warp_sum(t);
            if (threadIdx.x == 0) rs[r] = rsqrtf(t / (float)K + eps);
        }
    }
    const float4* g4 = reinterpret_cast<const float4*>(gain);
#pragma unroll
    for (int j = 0; j < PF_NORM_V; ++j) {
        const int i = threadIdx.x + j * PF_EW_THREADS;
        if (i < n4) {
            float4 w = v[j];
            const float4 gg = g4[i];
            w.x *= gg.x; w.y *= gg.y; w.z *= gg.z; w.w *= gg.w;
            split_store4(hi, lo, (size_t)r * K + (size_t)i * 4, w);
        }
    }
}

// planes of x[r] itself; grid = (rows, ceil(K / (4 * PF_EW_THREADS))), K and ldx multiples of 4
__global__ void __launch_bounds__(PF_EW_THREADS) pf_split_kernel(const float* x, int ldx, int K, __nv_bfloat16* hi, __nv_bfloat16* lo) {
    const int r = blockIdx.x;
    const int i = blockIdx.y * PF_EW_THREADS + threadIdx.x;
    if (i < (K >> 2)) split_store4(hi, lo, (size_t)r * K + (size_t)i * 4, *reinterpret_cast<const float4*>(x + (size_t)r * ldx + (size_t)i * 4));
}

// planes of SiLU(gate) * up; grid = (rows, ceil(F / (4 * PF_EW_THREADS))), F a multiple of 4
__global__ void __launch_bounds__(PF_EW_THREADS) pf_swiglu_split_kernel(const float* gate, const float* up, int F, __nv_bfloat16* hi, __nv_bfloat16* lo) {
    const int r = blockIdx.x;
    const int i = blockIdx.y * PF_EW_THREADS + threadIdx.x;
    if (i < (F >> 2)) {
        const size_t o = (size_t)r * F + (size_t)i * 4;
        const float4 gt = *reinterpret_cast<const float4*>(gate + o);
        const float4 u = *reinterpret_cast<const float4*>(up + o);
        split_store4(hi, lo, o, make_float4(silu_f(gt.x) * u.x, silu_f(gt.y) * u.y, silu_f(gt.z) * u.z, silu_f(gt.w) * u.w));
    }
}

// K (rotated) and V rows of a block of prompt rows -> cache, rounded to the storage type; grid = (rows, H)
template <typename WT>
__global__ void pf_rope_append_kernel(const Dev D, const float* qkv, int pos0, WT* kc, WT* vc) {
    const int r = blockIdx.x, hh = blockIdx.y, pos = pos0 + r;
    const int d = D.dm.d, hd = D.dm.hd, half = hd >> 1, H = D.dm.H, ps = D.dm.page_size;
    const float* src = qkv + (size_t)r * 3 * d + hh * hd;
    const int page = D.page_table[pos >> D.dm.ps_shift];
    const size_t base = (((size_t)page * H + hh) * ps + (pos & (ps - 1))) * hd;
    for (int e = threadIdx.x; e < half; e += blockDim.x) {
        float cs, sn; rope_cs(D, pos, e, cs, sn);
        const float k1 = src[d + e], k2 = src[d + e + half];
        kc[base + e] = float_to_wt<WT>(k1 * cs - k2 * sn);
        kc[base + e + half] = float_to_wt<WT>(k2 * cs + k1 * sn);
        vc[base + e] = float_to_wt<WT>(src[2 * d + e]);
        vc[base + e + half] = float_to_wt<WT>(src[2 * d + e + half]);
    }
}

}  // namespace kg
