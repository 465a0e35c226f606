// Device-side building blocks of the Kangaroo decode step for sm_100a.
//
// Everything here is written as __device__ "operators" that every CTA of a persistent,
// cooperatively launched grid executes in lock step: each operator splits its work by
// (cta, nctas) and a grid-wide barrier separates dependent operators.  The same operators are
// also wrapped one-by-one in small kernels for unit tests.
//
// Data flow is weight streaming: every weight byte is read exactly once per pass, straight from
// HBM into registers with 128-bit non-allocating loads, and consumed by tensor-core MMAs whose
// "M" side is the weight tile and whose "N" side is the 1..16 activation rows.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kg {

constexpr int M_MAX = 16;          // rows per pass
constexpr int NTHREADS = 512;      // threads per CTA
constexpr int NWARPS = NTHREADS / 32;
constexpr int S_CAP = 16;          // most KV splits per head
constexpr int ATT_TK = 64;         // keys per attention tile
constexpr int HD_MAX = 128;
constexpr int LIN_U = 4;           // k32-steps in flight per warp iteration
constexpr int XS_BUDGET = 168 * 1024;   // shared-memory bytes for staged activations
constexpr unsigned long long BARRIER_TIMEOUT_CLK = 6000000000ull;   // ~3 s at 1.9 GHz

enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_HEAD = 3 };
enum { ST_OK = 0, ST_TIMEOUT = -6 };

struct LayerW {
    const void* wqkv; const void* wo; const void* wgate; const void* wup; const void* wdown;
    const float* g1; const float* g2;
};

struct Dims {
    int L, d, H, hd, F, V, l;
    float eps, theta, logit_scale;
    int max_seq, page_size, n_pages, gamma_max, debug;
};

// Device-resident sequence / round state (one int-sized field per line of the method's notation).
struct State {
    int P;              // position of x_0 = tokens held by the shallow and deep KV caches
    int len_A;          // tokens held by the adapter's KV cache (P or P-1)
    int x0;             // the round's first token
    int pending;        // 1: a drafted unit awaits kg_verify
    int n_d;            // drafts kept this round
    int n_steps;        // adapter+head passes this round
    int M, k_acc, n_emit;
    int total;          // tokens in out_tokens (x_0 of prefill included)
    int rounds;
    int draft_steps_total, drafted_total, accepted_total;
    int status;         // 0 or a negative kg_status set by a device-side wait that gave up
    int timeout_where;
    int draft_tok[M_MAX];
    float conf[M_MAX];
    int emitted[M_MAX];
    int target[M_MAX];
};

struct Dev {
    Dims dm;
    const void* embed; const void* head; const float* g_final;
    const LayerW* layers;          // [L+1], index L = adapter
    void* kcache; void* vcache;    // [(L+1)][n_pages][H][page_size][hd]
    const int* page_table;         // [n_pages] logical -> physical page
    float* h;                      // [M_MAX][d] residual stream of the pass
    float* feat;                   // [M_MAX+1][d]: slot 0 = early feature of position P-1, slot 1+j = f_j
    float* abuf;                   // [2][d] adapter output rows
    float* qkv;                    // [M_MAX][3d]
    float* attn;                   // [M_MAX][d]
    float* act;                    // [M_MAX][F]
    float* att_po;                 // [M_MAX][H][S_CAP][hd] split partial outputs
    float* att_ml;                 // [M_MAX][H][S_CAP][2]  split partial (max, sum)
    unsigned* att_cnt;             // [H] arrival counters
    float4* head_part;             // [nctas][M_MAX] (zmax, sumexp, argmax bits, -)
    float* dbg_draft; float* dbg_verify;   // [M_MAX][V] each (debug only)
    int* out_tokens; int* S; int* round_log;   // [max_seq], [max_seq], [max_seq][4]
    const int* prompt;             // device copy of the prompt
    State* st;
    unsigned* bar;                 // grid barrier arrival counter (zeroed before every launch)
    double inv_freq[HD_MAX / 2];   // theta^(-2i/hd)
};

struct Ctx {
    int cta, nctas;
    unsigned bar_target;           // arrivals expected at the next barrier (thread 0 only)
    State* st; unsigned* bar;
    char* smem;
    bool grid;                     // false: single-operator test kernel, barriers are no-ops
};

// ------------------------------------------------------------------------------------ helpers

__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ldcg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ldcg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                               unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <typename WT> __device__ __forceinline__ float wt_to_float(WT v);
template <> __device__ __forceinline__ float wt_to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float wt_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename WT> __device__ __forceinline__ WT float_to_wt(float v);
template <> __device__ __forceinline__ float float_to_wt<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 float_to_wt<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename WT> __device__ __forceinline__ float4 load4_cg(const WT* p);
template <> __device__ __forceinline__ float4 load4_cg<float>(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
template <> __device__ __forceinline__ float4 load4_cg<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint2 r = __ldcg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
}

// (better, z, idx): larger z wins; on equal z the lower index wins.
__device__ __forceinline__ bool arg_better(float za, int ia, float zb, int ib) {
    return za > zb || (za == zb && ia < ib);
}

// ------------------------------------------------------------------------------------ grid barrier
// Monotonic arrival counter; every wait is bounded.  On expiry the kernel records KG_E_TIMEOUT in
// the state word and every CTA leaves at its next barrier.  Returns false when the grid must stop.
__device__ __forceinline__ bool grid_sync(Ctx& c, int where) {
    if (!c.grid) { __syncthreads(); return true; }
    __shared__ int s_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        c.bar_target += (unsigned)c.nctas;
        __threadfence();
        atomicAdd(c.bar, 1u);
        int ok = 1;
        long long t0 = clock64();
        unsigned spins = 0;
        while ((int)(ld_acquire_u32(c.bar) - c.bar_target) < 0) {
            if (((++spins) & 63u) == 0u) {
                if (*(volatile int*)&c.st->status != 0) { ok = 0; break; }
                if ((unsigned long long)(clock64() - t0) > BARRIER_TIMEOUT_CLK) {
                    atomicCAS(&c.st->status, 0, ST_TIMEOUT);
                    c.st->timeout_where = where;
                    ok = 0;
                    break;
                }
            }
        }
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

// ------------------------------------------------------------------------------------ RoPE
// cos / sin of pos * theta^(-2i/hd): the angle is formed and reduced to [-pi, pi] in double, the
// trigonometric functions are evaluated in fp32 on the reduced argument.
__device__ __forceinline__ void rope_cs(const Dev& D, int pos, int i, float& cs, float& sn) {
    double a = (double)pos * D.inv_freq[i];
    const double two_pi = 6.283185307179586476925286766559;
    double k = rint(a / two_pi);
    float r = (float)(a - k * two_pi);
    sincosf(r, &sn, &cs);
}

// ------------------------------------------------------------------------------------ linear operator
struct LinArgs {
    const void* W; const void* W2;   // [N, K]; W2 != null: SwiGLU pair (gate, up)
    int N, K;
    const float* x; int ldx; int M;  // activation rows (fp32, written earlier in this kernel)
    const float* gain; float eps;    // RMSNorm gain (null: no norm)
    const float* resid; int ldr;     // EPI_RESID
    float* out; int ldo;
    int epi;
    float scale;                     // EPI_HEAD: logit scale
    float4* head_part;               // EPI_HEAD: [nctas][M_MAX]
    float* logits_dbg; int ld_dbg;   // EPI_HEAD, optional
};

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + expf(-v)); }

// Running (max, argmax, sum exp) of one logit row, merged in a fixed order.
struct HeadStat { float zmax; float sum; int arg; };
__device__ __forceinline__ void head_merge(HeadStat& a, float zmax, float sum, int arg) {
    if (sum == 0.0f) return;
    if (a.sum == 0.0f) { a.zmax = zmax; a.sum = sum; a.arg = arg; return; }
    if (arg_better(zmax, arg, a.zmax, a.arg)) {
        a.sum = a.sum * expf(a.zmax - zmax) + sum;
        a.zmax = zmax; a.arg = arg;
    } else {
        a.sum = a.sum + sum * expf(zmax - a.zmax);
    }
}

// Tensor-core path, bf16 weights, 1 <= M <= 8*NT.  Swap-AB: the weight tile is the 16-row MMA
// operand, the activation rows are the 8 MMA columns.  A fragments come straight from global
// memory: lane (g, t) loads 16 contiguous bytes of weight row g and of row g+8; the k index is
// permuted identically for A and B so no shuffle or shared-memory staging of weights is needed.
// Activations are staged once per CTA in shared memory as bf16 hi + lo (x = hi + lo to ~2^-17),
// with the RMSNorm gain folded in; the 1/rms factor is applied in the epilogue.
template <int NT>
__device__ void lin_mma(const LinArgs& a, Ctx& c) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int M = a.M, K = a.K;
    const __nv_bfloat16* W = reinterpret_cast<const __nv_bfloat16*>(a.W);
    const __nv_bfloat16* W2 = reinterpret_cast<const __nv_bfloat16*>(a.W2);
    const bool dual = W2 != nullptr;

    const long long r0 = (long long)a.N * c.cta / c.nctas;
    const long long r1 = (long long)a.N * (c.cta + 1) / c.nctas;
    const int nr = (int)(r1 - r0);
    const int rpt = dual ? 8 : 16;                       // output rows (or gate/up pairs) per tile
    const int ntiles = (nr + rpt - 1) / rpt;
    const int nchunks = (ntiles + 3) / 4;

    // phases over K so that the staged activations fit
    int plen_max = (XS_BUDGET / (4 * M) - 32) & ~63;
    int nph = (K + plen_max - 1) / plen_max;
    int plen = (((K + nph - 1) / nph) + 63) & ~63;
    const int xstride = plen + 32;                       // bf16 elements; byte stride = 64 (mod 128)

    __nv_bfloat16* xs_hi = reinterpret_cast<__nv_bfloat16*>(c.smem);
    __nv_bfloat16* xs_lo = xs_hi + (size_t)M * xstride;
    float* red = reinterpret_cast<float*>(c.smem + XS_BUDGET);          // [2][NWARPS][NT][16][8]
    float* ssw = red + 2 * NWARPS * NT * 128;                           // [NWARPS][M_MAX]
    float* rs = ssw + NWARPS * M_MAX;                                   // [M_MAX]

    for (int i = tid; i < NWARPS * M_MAX; i += NTHREADS) ssw[i] = 0.0f;
    __syncthreads();

    HeadStat hs; hs.zmax = 0.f; hs.sum = 0.f; hs.arg = 0;               // EPI_HEAD: warp m tracks row m
    int buf = 0;
    bool rs_ready = false;

    for (int ch = 0; ch < nchunks; ++ch) {
        const int t0 = ch * 4;
        const int nt = min(4, ntiles - t0);
        const int n_ks = NWARPS / nt;
        const int my_tile = warp / n_ks, my_ks = warp % n_ks;
        const bool active = my_tile < nt;
        const __nv_bfloat16 *pA = nullptr, *pB = nullptr;
        if (active) {
            if (!dual) {
                long long ra = r0 + (long long)(t0 + my_tile) * 16 + g;
                if (ra < r1) pA = W + ra * K;
                if (ra + 8 < r1) pB = W + (ra + 8) * K;
            } else {
                long long f = r0 + (long long)(t0 + my_tile) * 8 + g;
                if (f < r1) { pA = W + f * K; pB = W2 + f * K; }
            }
        }
        float acc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }

        for (int ph = 0; ph < nph; ++ph) {
            const int p0 = ph * plen;
            const int len = min(plen, K - p0);
            if (nph > 1 || ch == 0) {
                if (nph > 1) __syncthreads();
                // stage x[:, p0:p0+len] * gain as bf16 hi / lo; accumulate sum of squares (first chunk only)
                for (int m = 0; m < M; ++m) {
                    float ss = 0.f;
                    const float* xr = a.x + (size_t)m * a.ldx + p0;
                    for (int u = tid; u < len / 8; u += NTHREADS) {
                        float4 v0 = ldcg_f4(xr + u * 8), v1 = ldcg_f4(xr + u * 8 + 4);
                        if (a.gain) {
                            ss += v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w
                                + v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
                            float4 g0 = ldcg_f4(a.gain + p0 + u * 8), g1 = ldcg_f4(a.gain + p0 + u * 8 + 4);
                            v0.x *= g0.x; v0.y *= g0.y; v0.z *= g0.z; v0.w *= g0.w;
                            v1.x *= g1.x; v1.y *= g1.y; v1.z *= g1.z; v1.w *= g1.w;
                        }
                        float f[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                        __align__(16) __nv_bfloat16 hi[8], lo[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            hi[e] = __float2bfloat16_rn(f[e]);
                            lo[e] = __float2bfloat16_rn(f[e] - __bfloat162float(hi[e]));
                        }
                        *reinterpret_cast<uint4*>(xs_hi + (size_t)m * xstride + u * 8) = *reinterpret_cast<uint4*>(hi);
                        *reinterpret_cast<uint4*>(xs_lo + (size_t)m * xstride + u * 8) = *reinterpret_cast<uint4*>(lo);
                    }
                    if (a.gain && ch == 0) {
                        ss = warp_sum(ss);
                        if (lane == 0) ssw[warp * M_MAX + m] += ss;
                    }
                }
                __syncthreads();
            }
            if (active) {
                const int steps = len / 32;
                const int sb = steps * my_ks / n_ks, se = steps * (my_ks + 1) / n_ks;
                for (int s = sb; s < se; s += LIN_U) {
                    uint4 wa[LIN_U], wb[LIN_U];
#pragma unroll
                    for (int u = 0; u < LIN_U; ++u) {
                        wa[u] = make_uint4(0, 0, 0, 0); wb[u] = make_uint4(0, 0, 0, 0);
                        if (s + u < se) {
                            const int k = p0 + (s + u) * 32 + 8 * t;
                            if (pA) wa[u] = ldg_stream16(pA + k);
                            if (pB) wb[u] = ldg_stream16(pB + k);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < LIN_U; ++u) {
                        if (s + u < se) {
                            const int kl = (s + u) * 32 + 8 * t;
#pragma unroll
                            for (int n = 0; n < NT; ++n) {
                                const int m = g + 8 * n;
                                uint4 xh = make_uint4(0, 0, 0, 0), xl = make_uint4(0, 0, 0, 0);
                                if (m < M) {
                                    xh = *reinterpret_cast<const uint4*>(xs_hi + (size_t)m * xstride + kl);
                                    xl = *reinterpret_cast<const uint4*>(xs_lo + (size_t)m * xstride + kl);
                                }
                                mma_bf16_16816(acc[n], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xh.x, xh.y);
                                mma_bf16_16816(acc[n], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xh.z, xh.w);
                                mma_bf16_16816(acc[n], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xl.x, xl.y);
                                mma_bf16_16816(acc[n], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xl.z, xl.w);
                            }
                        }
                    }
                }
            }
        }
        // partial sums of this (tile, k-slice) item
        float* rb = red + (size_t)buf * NWARPS * NT * 128;
        if (active) {
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                float* r = rb + ((size_t)warp * NT + n) * 128;
                *reinterpret_cast<float2*>(r + g * 8 + 2 * t) = make_float2(acc[n][0], acc[n][1]);
                *reinterpret_cast<float2*>(r + (g + 8) * 8 + 2 * t) = make_float2(acc[n][2], acc[n][3]);
            }
        }
        __syncthreads();
        if (!rs_ready) {      // 1/rms per row, summed over warps in a fixed order (same value in every thread)
            rs_ready = true;
            if (tid < M_MAX) {
                float r = 1.0f;
                if (a.gain && tid < M) {
                    float ss = 0.f;
                    for (int w = 0; w < NWARPS; ++w) ss += ssw[w * M_MAX + tid];
                    r = rsqrtf(ss / (float)K + a.eps);
                }
                rs[tid] = r;
            }
            __syncthreads();
        }
        // value of (tile-local row r16, activation row m) summed over the k-slices in order
        auto reduced = [&](int tile, int r16, int m) -> float {
            const float* r = rb + ((size_t)(tile * n_ks) * NT + (m >> 3)) * 128 + r16 * 8 + (m & 7);
            float v = 0.f;
            for (int ks = 0; ks < n_ks; ++ks) v += r[(size_t)ks * NT * 128];
            return v;
        };
        if (a.epi == EPI_SWIGLU) {
            const int nf = min(nt * 8, nr - t0 * 8);
            for (int idx = tid; idx < nf * M; idx += NTHREADS) {
                const int fl = idx % nf, m = idx / nf;
                const float vg = reduced(fl >> 3, fl & 7, m) * rs[m];
                const float vu = reduced(fl >> 3, (fl & 7) + 8, m) * rs[m];
                a.out[(size_t)m * a.ldo + r0 + t0 * 8 + fl] = silu_f(vg) * vu;
            }
        } else if (a.epi == EPI_HEAD) {
            const int nrow = min(nt * 16, nr - t0 * 16);
            if (warp < M) {
                const int m = warp;
                float zl[2]; int il[2];
                float zm = -INFINITY; int im = 0x7fffffff;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int r = lane + 32 * q;
                    zl[q] = -INFINITY; il[q] = 0x7fffffff;
                    if (r < nrow) {
                        zl[q] = reduced(r >> 4, r & 15, m) * rs[m] * a.scale;
                        il[q] = (int)(r0 + t0 * 16 + r);
                        if (a.logits_dbg) a.logits_dbg[(size_t)m * a.ld_dbg + il[q]] = zl[q];
                        if (arg_better(zl[q], il[q], zm, im)) { zm = zl[q]; im = il[q]; }
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    float z2 = __shfl_xor_sync(0xffffffffu, zm, o);
                    int i2 = __shfl_xor_sync(0xffffffffu, im, o);
                    if (arg_better(z2, i2, zm, im)) { zm = z2; im = i2; }
                }
                float e = 0.f;
#pragma unroll
                for (int q = 0; q < 2; ++q) if (lane + 32 * q < nrow) e += expf(zl[q] - zm);
                e = warp_sum(e);
                head_merge(hs, zm, e, im);
            }
        } else {
            const int nrow = min(nt * 16, nr - t0 * 16);
            for (int idx = tid; idx < nrow * M; idx += NTHREADS) {
                const int r = idx % nrow, m = idx / nrow;
                float v = reduced(r >> 4, r & 15, m) * rs[m];
                const size_t row = (size_t)(r0 + t0 * 16 + r);
                if (a.epi == EPI_RESID) v += ldcg_f(a.resid + (size_t)m * a.ldr + row);
                a.out[(size_t)m * a.ldo + row] = v;
            }
        }
        buf ^= 1;
    }
    if (a.epi == EPI_HEAD && warp < M && lane == 0)
        a.head_part[(size_t)c.cta * M_MAX + warp] = make_float4(hs.zmax, hs.sum, __int_as_float(hs.arg), 0.f);
    __syncthreads();
}

// Plain path for any storage type (used for fp32 models and as a cross-check of the tensor-core
// path): activations staged in shared memory as fp32, one output row per warp at a time.
template <typename WT>
__device__ void lin_simple(const LinArgs& a, Ctx& c) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = a.M, K = a.K;
    const WT* W = reinterpret_cast<const WT*>(a.W);
    const WT* W2 = reinterpret_cast<const WT*>(a.W2);
    const bool dual = W2 != nullptr;
    float* xs = reinterpret_cast<float*>(c.smem);                        // [M][K]
    float* rs = reinterpret_cast<float*>(c.smem + XS_BUDGET);            // [M_MAX]
    float* wst = rs + M_MAX;                                             // [NWARPS][M_MAX][3] head stats

    for (int m = warp; m < M; m += NWARPS) {
        float ss = 0.f;
        for (int k = lane; k < K; k += 32) {
            float v = ldcg_f(a.x + (size_t)m * a.ldx + k);
            ss += v * v;
            xs[(size_t)m * K + k] = a.gain ? v * ldcg_f(a.gain + k) : v;
        }
        ss = warp_sum(ss);
        if (lane == 0) rs[m] = a.gain ? rsqrtf(ss / (float)K + a.eps) : 1.0f;
    }
    __syncthreads();

    HeadStat hs; hs.zmax = 0.f; hs.sum = 0.f; hs.arg = 0;               // lane m tracks row m
    for (long long row = (long long)c.cta * NWARPS + warp; row < a.N; row += (long long)c.nctas * NWARPS) {
        float acc[M_MAX], acc2[M_MAX];
#pragma unroll
        for (int m = 0; m < M_MAX; ++m) { acc[m] = 0.f; acc2[m] = 0.f; }
        const WT* wr = W + (size_t)row * K;
        const WT* wr2 = dual ? W2 + (size_t)row * K : nullptr;
        for (int k = lane; k < K; k += 32) {
            const float w = wt_to_float<WT>(wr[k]);
            const float w2 = dual ? wt_to_float<WT>(wr2[k]) : 0.f;
#pragma unroll
            for (int m = 0; m < M_MAX; ++m) {
                if (m < M) {
                    const float xv = xs[(size_t)m * K + k];
                    acc[m] = fmaf(w, xv, acc[m]);
                    if (dual) acc2[m] = fmaf(w2, xv, acc2[m]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < M_MAX; ++m) {
            if (m < M) {
                float v = warp_sum(acc[m]) * rs[m];
                float v2 = dual ? warp_sum(acc2[m]) * rs[m] : 0.f;
                if (a.epi == EPI_HEAD) {
                    v *= a.scale;
                    if (lane == 0 && a.logits_dbg) a.logits_dbg[(size_t)m * a.ld_dbg + row] = v;
                    if (lane == m) head_merge(hs, v, 1.0f, (int)row);
                } else if (lane == 0) {
                    if (a.epi == EPI_SWIGLU) v = silu_f(v) * v2;
                    if (a.epi == EPI_RESID) v += ldcg_f(a.resid + (size_t)m * a.ldr + row);
                    a.out[(size_t)m * a.ldo + row] = v;
                }
            }
        }
    }
    if (a.epi == EPI_HEAD) {
        if (lane < M) {
            wst[(warp * M_MAX + lane) * 3 + 0] = hs.zmax;
            wst[(warp * M_MAX + lane) * 3 + 1] = hs.sum;
            wst[(warp * M_MAX + lane) * 3 + 2] = __int_as_float(hs.arg);
        }
        __syncthreads();
        if (tid < M) {
            HeadStat tot; tot.zmax = 0.f; tot.sum = 0.f; tot.arg = 0;
            for (int w = 0; w < NWARPS; ++w)
                head_merge(tot, wst[(w * M_MAX + tid) * 3 + 0], wst[(w * M_MAX + tid) * 3 + 1],
                           __float_as_int(wst[(w * M_MAX + tid) * 3 + 2]));
            a.head_part[(size_t)c.cta * M_MAX + tid] = make_float4(tot.zmax, tot.sum, __int_as_float(tot.arg), 0.f);
        }
    }
    __syncthreads();
}

template <typename WT> struct LinDispatch;
template <> struct LinDispatch<float> {
    static __device__ __forceinline__ void run(const LinArgs& a, Ctx& c, bool) { lin_simple<float>(a, c); }
};
template <> struct LinDispatch<__nv_bfloat16> {
    static __device__ __forceinline__ void run(const LinArgs& a, Ctx& c, bool force_simple) {
        if (force_simple || (a.K & 31) != 0) lin_simple<__nv_bfloat16>(a, c);
        else if (a.M <= 8) lin_mma<1>(a, c);
        else lin_mma<2>(a, c);
    }
};

// Merge the per-CTA head partials of row m (identical result in every CTA: fixed order).
__device__ __forceinline__ void head_final(const float4* part, int nctas, int m, int& tok, float& p) {
    HeadStat tot; tot.zmax = 0.f; tot.sum = 0.f; tot.arg = 0;
    for (int cta = 0; cta < nctas; ++cta) {
        float4 v = __ldcg(part + (size_t)cta * M_MAX + m);
        head_merge(tot, v.x, v.y, __float_as_int(v.z));
    }
    tok = tot.arg;
    p = 1.0f / tot.sum;
}

// ------------------------------------------------------------------------------------ attention operator
struct AttArgs {
    const float* qkv;      // [M][3d] raw q, k, v rows of this pass
    int M, pos0;           // rows sit at positions pos0 .. pos0+M-1; row i sees keys 0 .. pos0+i
    void* kc; void* vc;    // this layer's cache: [n_pages][H][page_size][hd]
    float* out;            // [M][d]
};

// One work item = (head, KV split).  Keys come from the paged cache; the rows of this pass are
// rotated (RoPE), rounded to the cache's storage type and appended to the cache by the item whose
// key range contains them, then read back like any other key.  Every split writes a partial
// (max, sum, o); the last split of a head to arrive merges them in split order.
template <typename WT>
__device__ void attention_op(const Dev& D, const AttArgs& a, Ctx& c) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = D.dm.H, hd = D.dm.hd, d = D.dm.d, ps = D.dm.page_size;
    const int M = a.M, pos0 = a.pos0;
    const int T = pos0 + M;
    const int half = hd >> 1;
    int S = min(min(S_CAP, max(1, (2 * c.nctas) / H)), (T + ATT_TK - 1) / ATT_TK);
    const int chunk = (T + S - 1) / S;
    const float sc = rsqrtf((float)hd);
    WT* kc = reinterpret_cast<WT*>(a.kc);
    WT* vc = reinterpret_cast<WT*>(a.vc);

    float* qs = reinterpret_cast<float*>(c.smem);                  // [M_MAX][HD_MAX]
    float* Ks = qs + M_MAX * HD_MAX;                               // [ATT_TK][hd+4]
    float* Vs = Ks + ATT_TK * (HD_MAX + 4);                        // [ATT_TK][hd]
    float* Ss = Vs + ATT_TK * HD_MAX;                              // [M_MAX][ATT_TK]
    float* mrun = Ss + M_MAX * ATT_TK;                             // [M_MAX] running max
    float* lrun = mrun + M_MAX;                                    // [M_MAX] running sum
    float* corr = lrun + M_MAX;                                    // [M_MAX]
    __shared__ int s_last;
    const int kstr = hd + 4;
    const int rgs = NTHREADS / hd;                                 // row groups in the PV phase
    const int e_pv = tid % hd, rg_pv = tid / hd;
    constexpr int PV_R = 4;                                        // rows per thread in PV (rgs >= 4)

    for (int item = c.cta; item < H * S; item += c.nctas) {
        const int hh = item / S, s = item % S;
        const int kb = s * chunk, ke = min(T, kb + chunk);
        __syncthreads();
        // q rows: RoPE, pre-scaled by 1/sqrt(hd)
        for (int idx = tid; idx < M * half; idx += NTHREADS) {
            const int i = idx / half, e = idx % half;
            float cs, sn; rope_cs(D, pos0 + i, e, cs, sn);
            const float x1 = ldcg_f(a.qkv + (size_t)i * 3 * d + hh * hd + e);
            const float x2 = ldcg_f(a.qkv + (size_t)i * 3 * d + hh * hd + e + half);
            qs[i * HD_MAX + e] = (x1 * cs - x2 * sn) * sc;
            qs[i * HD_MAX + e + half] = (x2 * cs + x1 * sn) * sc;
        }
        // append this pass's K / V rows that fall into my key range
        {
            const int nb = max(kb, pos0), ne = ke;
            for (int idx = tid; idx < (ne - nb) * half; idx += NTHREADS) {
                const int pos = nb + idx / half, e = idx % half, i = pos - pos0;
                float cs, sn; rope_cs(D, pos, e, cs, sn);
                const float* src = a.qkv + (size_t)i * 3 * d + hh * hd;
                const float k1 = ldcg_f(src + d + e), k2 = ldcg_f(src + d + e + half);
                const size_t base = (((size_t)D.page_table[pos / ps] * H + hh) * ps + pos % ps) * hd;
                kc[base + e] = float_to_wt<WT>(k1 * cs - k2 * sn);
                kc[base + e + half] = float_to_wt<WT>(k2 * cs + k1 * sn);
                vc[base + e] = float_to_wt<WT>(ldcg_f(src + 2 * d + e));
                vc[base + e + half] = float_to_wt<WT>(ldcg_f(src + 2 * d + e + half));
            }
        }
        if (tid < M_MAX) { mrun[tid] = -INFINITY; lrun[tid] = 0.f; }
        float o[PV_R];
#pragma unroll
        for (int r = 0; r < PV_R; ++r) o[r] = 0.f;
        __syncthreads();

        for (int tb = kb; tb < ke; tb += ATT_TK) {
            const int nk = min(ATT_TK, ke - tb);
            // stage K and V tiles as fp32
            for (int idx = tid; idx < nk * (hd / 4); idx += NTHREADS) {
                const int j = idx / (hd / 4), e4 = (idx % (hd / 4)) * 4;
                const int pos = tb + j;
                const size_t base = (((size_t)D.page_table[pos / ps] * H + hh) * ps + pos % ps) * hd + e4;
                const float4 kv = load4_cg<WT>(kc + base), vv = load4_cg<WT>(vc + base);
                *reinterpret_cast<float4*>(Ks + j * kstr + e4) = kv;
                *reinterpret_cast<float4*>(Vs + j * hd + e4) = vv;
            }
            __syncthreads();
            // scores: thread (key j, row group) -> rows i = rgq, rgq + 8
            {
                const int j = tid % ATT_TK, rgq = tid / ATT_TK;          // 8 row groups
                float s0 = 0.f, s1 = 0.f;
                const bool r0v = rgq < M, r1v = rgq + 8 < M;
                if (j < nk && r0v) {
                    const float* kr = Ks + j * kstr;
                    const float* q0 = qs + rgq * HD_MAX;
                    const float* q1 = qs + (rgq + 8) * HD_MAX;
                    for (int e4 = 0; e4 < hd; e4 += 4) {
                        const float4 kv = *reinterpret_cast<const float4*>(kr + e4);
                        const float4 a0 = *reinterpret_cast<const float4*>(q0 + e4);
                        s0 = fmaf(kv.x, a0.x, fmaf(kv.y, a0.y, fmaf(kv.z, a0.z, fmaf(kv.w, a0.w, s0))));
                        if (r1v) {
                            const float4 a1 = *reinterpret_cast<const float4*>(q1 + e4);
                            s1 = fmaf(kv.x, a1.x, fmaf(kv.y, a1.y, fmaf(kv.z, a1.z, fmaf(kv.w, a1.w, s1))));
                        }
                    }
                }
                const int pos = tb + j;
                if (r0v) Ss[rgq * ATT_TK + j] = (j < nk && pos <= pos0 + rgq) ? s0 : -INFINITY;
                if (r1v) Ss[(rgq + 8) * ATT_TK + j] = (j < nk && pos <= pos0 + rgq + 8) ? s1 : -INFINITY;
            }
            __syncthreads();
            // online softmax bookkeeping: warp i owns row i
            if (warp < M) {
                const int i = warp;
                const float v0 = Ss[i * ATT_TK + lane], v1 = Ss[i * ATT_TK + lane + 32];
                const float mo = mrun[i];
                const float mn = fmaxf(mo, warp_max(fmaxf(v0, v1)));
                float p0 = 0.f, p1 = 0.f, cf = 1.f;
                if (mn != -INFINITY) {
                    p0 = expf(v0 - mn); p1 = expf(v1 - mn);
                    cf = (mo == -INFINITY) ? 0.f : expf(mo - mn);
                }
                Ss[i * ATT_TK + lane] = p0; Ss[i * ATT_TK + lane + 32] = p1;
                const float ps_ = warp_sum(p0 + p1);
                if (lane == 0) { lrun[i] = lrun[i] * cf + ps_; mrun[i] = mn; corr[i] = cf; }
            }
            __syncthreads();
            // o += P V : thread (element e, row group) -> rows i = rg_pv + rgs * r
            if (rg_pv < rgs) {
#pragma unroll
                for (int r = 0; r < PV_R; ++r) {
                    const int i = rg_pv + rgs * r;
                    if (i < M) {
                        float accv = o[r] * corr[i];
                        const float* pr = Ss + i * ATT_TK;
                        for (int j = 0; j < nk; ++j) accv = fmaf(pr[j], Vs[j * hd + e_pv], accv);
                        o[r] = accv;
                    }
                }
            }
            __syncthreads();
        }
        // partials
        if (rg_pv < rgs) {
#pragma unroll
            for (int r = 0; r < PV_R; ++r) {
                const int i = rg_pv + rgs * r;
                if (i < M) D.att_po[(((size_t)i * H + hh) * S_CAP + s) * hd + e_pv] = o[r];
            }
        }
        if (tid < M) {
            D.att_ml[(((size_t)tid * H + hh) * S_CAP + s) * 2 + 0] = mrun[tid];
            D.att_ml[(((size_t)tid * H + hh) * S_CAP + s) * 2 + 1] = lrun[tid];
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned prev = atomicAdd(D.att_cnt + hh, 1u);
            s_last = (prev == (unsigned)(S - 1));
            if (s_last) { D.att_cnt[hh] = 0u; __threadfence(); }
        }
        __syncthreads();
        if (s_last) {
            for (int idx = tid; idx < M * hd; idx += NTHREADS) {
                const int i = idx / hd, e = idx % hd;
                const float* ml = D.att_ml + ((size_t)i * H + hh) * S_CAP * 2;
                float mx = -INFINITY;
                for (int q = 0; q < S; ++q) mx = fmaxf(mx, ldcg_f(ml + q * 2));
                float den = 0.f, num = 0.f;
                for (int q = 0; q < S; ++q) {
                    const float mq = ldcg_f(ml + q * 2);
                    if (mq == -INFINITY) continue;
                    const float w = expf(mq - mx);
                    den += ldcg_f(ml + q * 2 + 1) * w;
                    num += ldcg_f(D.att_po + (((size_t)i * H + hh) * S_CAP + q) * hd + e) * w;
                }
                a.out[(size_t)i * d + hh * hd + e] = num / den;
            }
        }
    }
    __syncthreads();
}

__host__ __device__ inline size_t smem_bytes_needed() {
    size_t lin = (size_t)XS_BUDGET + (2 * NWARPS * 2 * 128 + NWARPS * M_MAX + M_MAX + NWARPS * M_MAX * 3 + 64) * sizeof(float);
    size_t att = (size_t)(M_MAX * HD_MAX + ATT_TK * (HD_MAX + 4) + ATT_TK * HD_MAX + M_MAX * ATT_TK + 3 * M_MAX) * sizeof(float);
    return lin > att ? lin : att;
}

}  // namespace kg
