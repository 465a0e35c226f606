// Device-side building blocks of the Kangaroo decode step for sm_100a.
//
// Everything here is written as __device__ "operators" that every CTA of a persistent,
// cooperatively launched grid executes in lock step: each operator splits its work by
// (cta, nctas) and a grid-wide barrier separates dependent operators.  The same operators are
// also wrapped one-by-one in small kernels for unit tests.
//
// A CTA has 8 consumer warps and one producer warp.  The decode step is bound by HBM bandwidth:
// every weight byte is read exactly once per pass.  The producer warp streams this CTA's share of
// every weight matrix of a pass through a ring of shared-memory slots with bulk asynchronous
// copies (cp.async.bulk + mbarrier transaction counts); because weights do not depend on
// activations it runs ahead of the consumers across operator boundaries and grid barriers, so HBM
// stays busy while the consumers synchronise.  The consumers read weight tiles with ldmatrix and
// feed tensor-core MMAs whose "M" side is the weight tile and whose "N" side is the 1..16
// activation rows (activations split into bf16 hi + lo so that the product keeps fp32 accuracy).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kg {

constexpr int M_MAX = 16;          // rows per pass
constexpr int NTHREADS = 256;      // consumer threads per CTA
constexpr int NWARPS = NTHREADS / 32;
constexpr int BLOCK_THREADS = NTHREADS + 32;   // + the producer warp (warp index NWARPS)
// The decode kernel is launched with a whole warpgroup behind the consumers (warp NWARPS is the producer, the other
// three leave at once): registers are handed out per warpgroup, and the producer's warpgroup gives most of its share
// to the two consumer warpgroups at kernel start (setmaxnreg).  The pool is what the launch allocated: 384 threads x
// 168 registers = 64512; a request beyond it would block forever, so the budgets below are checked against it.
constexpr int DECODE_THREADS = NTHREADS + 128;
constexpr int LAUNCH_REGS = 168;                  // 65536 / 384, rounded down to the allocation unit of 8
constexpr int CONSUMER_REGS = 216, PRODUCER_REGS = 56;
static_assert(NTHREADS * CONSUMER_REGS + 128 * PRODUCER_REGS <= DECODE_THREADS * LAUNCH_REGS, "register budgets exceed the CTA's pool");
static_assert(DECODE_THREADS * (LAUNCH_REGS + 8) > 65536, "LAUNCH_REGS is not what a launch of DECODE_THREADS threads gets");
constexpr int S_CAP = 16;          // most KV splits per head
constexpr int HD_MAX = 128;

// weight ring: RING slots of ST_ROWS weight rows x ST_K k-elements (bf16); rows are padded by 16
// bytes so that the eight row addresses of an ldmatrix fall into distinct bank groups
constexpr int RING = 6;
constexpr int ST_ROWS = 8;
constexpr int ST_K = 2048;
constexpr int ST_ROW_BYTES = ST_K * 2 + 16;
constexpr int SLOT_BYTES = ST_ROWS * ST_ROW_BYTES;
constexpr int CTRL_BYTES = 3072;
constexpr int OP_TABLE_BYTES = 1024;                    // struct OpTable: the operator arguments of one layer
constexpr int RING_OFF = CTRL_BYTES;
constexpr int WORK_OFF = RING_OFF + RING * SLOT_BYTES;
constexpr int SMEM_TOTAL = 232448;                      // 227 KB, the most one CTA may own
constexpr int WORK_BYTES = SMEM_TOTAL - WORK_OFF;       // activations, reductions, attention tiles
constexpr int SC_ROWS = 256;                            // rows whose accumulators live in shared memory at once
// the plain path never runs beside the streamed one in a launch, so it stages its activations over the ring too
constexpr int SIMPLE_XS_BYTES = SMEM_TOTAL - RING_OFF - 4096;

constexpr int BAR_RELEASE = 32;                          // word index of the grid barrier's release word (its own 128-byte line)
constexpr int BAR_BYTES = 256;
constexpr unsigned long long WAIT_TIMEOUT_CLK = 6000000000ull;   // default budget of a device-side wait: ~3 s at 1.9 GHz

enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2, EPI_HEAD = 3 };
enum { ST_OK = 0, ST_TIMEOUT = -6, ST_INTERNAL = -8 };

struct LayerW {
    const void* wqkv; const void* wo; const void* wgate; const void* wup; const void* wdown;
    const float* g1; const float* g2;
};

struct Dims {
    int L, d, H, hd, F, V, l;
    float eps, theta, logit_scale;
    int max_seq, page_size, n_pages, gamma_max, debug;
    int n_phys;         // physical pages behind the page table (page numbers must lie below it)
    int ps_shift;       // log2(page_size): page sizes are powers of two
    int stream;         // 1: linear operators take the streamed tensor-core path (bf16, d and F multiples of 16)
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
    // packed copies (streamed path; row = 4 bytes per element) and per-CTA sums of squares [row][nctas]
    unsigned char* hA_pk;          // [M_MAX][d]   residual stream scaled for the next QKV / the LM head
    unsigned char* hB_pk;          // [M_MAX][d]   residual stream after attention scaled for the SwiGLU pair
    unsigned char* attn_pk;        // [M_MAX][d]
    unsigned char* act_pk;         // [M_MAX][F]
    unsigned char* featA_pk;       // [M_MAX+1][d] early features scaled by the adapter's input gain
    unsigned char* featD_pk;       // [M_MAX+1][d] early features scaled by the first deep layer's gain
    unsigned char* abuf_pk;        // [2][d]       adapter output scaled by its last gain
    float* ssq_hA; float* ssq_hB;  // [M_MAX][nctas]
    float* ssq_feat;               // [M_MAX+1][nctas]
    float* ssq_abuf;               // [2][nctas]
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

// Per-CTA control block at the start of shared memory.
struct Ctrl {
    unsigned long long full[RING];     // producer -> consumers: slot filled (transaction count)
    unsigned long long empty[RING];    // consumers -> producer: slot drained (one arrival per consumer warp)
    unsigned long long mail;           // consumers -> producer: head_tok / head_p hold a new result
    int abort;                         // a bounded wait of this CTA gave up
    int sync_ok;
    int att_last;
    int head_tok[M_MAX];
    float head_p[M_MAX];
    // operator arguments of a whole layer (struct OpTable), written once per layer by one thread of each role and
    // read by all of its threads (kept here rather than on the per-thread stack, which the small L1 left beside
    // 227 KB of shared memory cannot hold)
    alignas(16) unsigned char tab_cons[OP_TABLE_BYTES];
    alignas(16) unsigned char tab_prod[OP_TABLE_BYTES];
    // the per-role context (struct Ctx): one copy for the consumers, one for the producer warp
    alignas(16) unsigned char ctx_cons[128];
    alignas(16) unsigned char ctx_prod[128];
};
static_assert(sizeof(Ctrl) <= CTRL_BYTES - 16, "control block too large");

// State of one role (consumers / producer warp) of the CTA.  It lives in shared memory: every thread of the role
// holds the same values, updates are the same in all of them, and between operators they are ordered by the
// role's barriers; reading it never touches the per-thread stack.
struct Ctx {
    int cta, nctas;
    unsigned bar_target;           // arrivals expected at the next grid barrier (thread 0 only)
    unsigned long long wait_clk;   // clocks after which a wait of this launch gives up
    State* st; unsigned* bar;
    int skip_arrival;              // test hook: 1 + index of the CTA that leaves out its first grid-barrier arrival (0: none)
    char* smem;
    Ctrl* ctl;
    bool grid;                     // false: single-operator test kernel, grid barriers are CTA barriers
    bool producer;                 // this thread belongs to the producer warp
    int slot; unsigned phase;      // ring cursor of this thread's role
    unsigned issued;               // producer: stages issued so far
    unsigned mail_phase;           // producer: parity of the next result it waits for
};

// ------------------------------------------------------------------------------------ helpers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ldcg_f(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float2 ldcg_f2(const float* p) { return __ldcg(reinterpret_cast<const float2*>(p)); }
__device__ __forceinline__ float4 ldcg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// barrier among the consumer warps only (the producer warp never takes part)
__device__ __forceinline__ void cta_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NTHREADS) : "memory"); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// global -> shared bulk copy; bytes and both addresses are multiples of 16.  `policy` is an L2 cache policy made by
// l2_evict_first(): weights are read once per pass, so their lines are the first to go, and what the pass re-reads
// (activations, K/V of the draft layers, barrier words) stays in L2 while 1-65 GB of weights stream past it.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src, unsigned bytes, unsigned long long* bar, unsigned long long policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ unsigned long long l2_evict_first() {
    unsigned long long p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// The top bit of the grid barrier's arrival counter tells every CTA that some wait has given up: they learn it from
// the word they poll anyway, without a second load.
constexpr unsigned BAR_ABORT = 0x80000000u;       // the host bounds a launch's arrivals below 2^31 (max_seq check)
__device__ __forceinline__ void record_timeout(Ctx& c, int where) {
    *(volatile int*)&c.ctl->abort = 1;
    if (c.st) {
        atomicCAS(&c.st->status, 0, ST_TIMEOUT);
        c.st->timeout_where = where;
    }
    if (c.grid && c.bar) atomicOr(c.bar, BAR_ABORT);
}

// Bounded wait on an mbarrier phase.  Returns false when this CTA has given up (here or elsewhere).
__device__ __forceinline__ bool mbar_wait(Ctx& c, unsigned long long* bar, unsigned parity, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        // the producer warp shares an issue port with two consumer warps: it backs off instead of spinning
        if (c.producer) __nanosleep(200);
        if (((++spins) & 63u) == 0u) {
            if (*(volatile int*)&c.ctl->abort) return false;
            if ((unsigned long long)(clock64() - t0) > c.wait_clk) { record_timeout(c, where); return false; }
        }
    }
    return true;
}

__device__ __forceinline__ void ldmatrix_x4(unsigned (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
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

// ------------------------------------------------------------------------------------ CTA set-up
// Called by every thread of the CTA at kernel start; returns the context of the thread's role.
__device__ __forceinline__ Ctx& ctx_init(char* smem, State* st, unsigned* bar, bool grid,
                                         unsigned long long wait_clk = WAIT_TIMEOUT_CLK, int skip_arrival = 0) {
    static_assert(sizeof(Ctx) <= 128, "context slot too small");
    Ctrl* ctl = reinterpret_cast<Ctrl*>(smem);
    const bool producer = threadIdx.x >= NTHREADS;
    Ctx& c = *reinterpret_cast<Ctx*>(producer ? ctl->ctx_prod : ctl->ctx_cons);
    if (threadIdx.x == 0 || threadIdx.x == NTHREADS) {
        c.cta = blockIdx.x; c.nctas = gridDim.x; c.bar_target = 0; c.st = st; c.bar = bar; c.smem = smem;
        c.wait_clk = wait_clk; c.skip_arrival = skip_arrival;
        c.ctl = ctl; c.grid = grid;
        c.producer = producer;
        c.slot = 0; c.phase = 0; c.issued = 0; c.mail_phase = 0;
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < RING; ++i) { mbar_init(&ctl->full[i], 1); mbar_init(&ctl->empty[i], NWARPS); }
        mbar_init(&ctl->mail, 1);
        ctl->abort = 0; ctl->sync_ok = 1; ctl->att_last = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    return c;
}

// ------------------------------------------------------------------------------------ grid barrier
// Consumer threads only.  Monotonic arrival counter; every wait is bounded.  On expiry the kernel
// records KG_E_TIMEOUT in the state word and every CTA leaves at its next barrier.  Returns false
// when the grid must stop (the same value in every consumer thread of the CTA).
__device__ __forceinline__ bool grid_sync(Ctx& c, int where) {
    if (!c.grid) { cta_sync(); return *(volatile int*)&c.ctl->abort == 0; }
    cta_sync();
    if (threadIdx.x == 0) {
        // bar[0] counts arrivals (monotonic over the launch, below 2^31: the host bounds max_seq accordingly): one
        // release-add, then poll until every CTA has arrived or the abort bit appears
        c.bar_target += (unsigned)c.nctas;
        const unsigned gen = c.bar_target;
        if (c.skip_arrival == c.cta + 1) c.skip_arrival = 0;        // test hook: this arrival never happens
        else asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(c.bar) : "memory");
        int ok = 1;
        {
            const long long t0 = clock64();
            unsigned spins = 0;
            while (true) {
                const unsigned v = ld_acquire_u32(c.bar);
                if (v & BAR_ABORT) { ok = 0; break; }
                if (v >= gen) break;
                if (((++spins) & 63u) == 0u) {
                    if ((unsigned long long)(clock64() - t0) > c.wait_clk) { record_timeout(c, where); ok = 0; break; }
                }
            }
        }
        if (!ok) *(volatile int*)&c.ctl->abort = 1;          // lets the producer warp leave its waits
        c.ctl->sync_ok = ok;
    }
    cta_sync();
    return *(volatile int*)&c.ctl->sync_ok != 0;
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
// A packed copy of activation rows: the row is cut into k16 blocks of 64 bytes; the 16 bytes at
// blk*64 + tt*16 hold {hi(k), hi(k+8), lo(k), lo(k+8)} for k = 16 blk + 2 tt, each a pair of bf16
// (elements k, k+1) with x * gain = hi + lo.  This is the B operand fragment order of the MMA, so a
// consumer lane fetches its fragments with plain 8- or 16-byte loads.  The operator that produces a
// row writes it once, in this form, for the operator that reads it.
struct PkOut { const float* gain; unsigned char* ptr; };   // gain == null: unscaled

// byte offset of the hi half of element k inside a packed row; the lo half sits 8 bytes further
__device__ __forceinline__ size_t pk_off(int k) {
    return (size_t)(k >> 4) * 64 + (size_t)(((k & 7) >> 1) * 16 + ((k >> 3) & 1) * 4 + (k & 1) * 2);
}
__device__ __forceinline__ void pk_store(unsigned char* row, int k, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
    unsigned char* p = row + pk_off(k);
    *reinterpret_cast<__nv_bfloat16*>(p) = h;
    *reinterpret_cast<__nv_bfloat16*>(p + 8) = l;
}

struct LinArgs {
    const void* W; const void* W2;   // [N, K]; W2 != null: SwiGLU pair (gate, up)
    int N, K;
    int M;                           // activation rows
    const float* x; int ldx;         // plain path: fp32 rows (written earlier in this kernel)
    const float* gain; float eps;    // RMSNorm gain of the input (null: no norm)
    const unsigned char* xpk; int ldpk;   // streamed path: packed rows, already multiplied by the gain; bytes per row
    const float* ssq_in;             // streamed path with norm: [M][nctas] partial sums of squares of the input rows
    const float* resid; int ldr;     // EPI_RESID
    float* out; int ldo;             // fp32 output rows (streamed path: nullable)
    int epi;
    float scale;                     // EPI_HEAD: logit scale
    float4* head_part;               // EPI_HEAD: [nctas][M_MAX]
    float* logits_dbg; int ld_dbg;   // EPI_HEAD, optional
    PkOut pk[2]; int ldpk_out;       // streamed path: packed copies of the output rows for the operators that read them
    float* ssq_out;                  // streamed path: [M][nctas] partial sums of squares of the output rows (nullable)
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

// ---- streamed tensor-core path (bf16 weights, K a multiple of 16) -----------------------------------
//
// Work split.  The CTA owns a contiguous range of "units": output rows, or for the SwiGLU pair
// gate/up feature pairs.  A stage of the ring holds 8 weight rows (for the pair: the 8 gate rows of
// a feature group, then in the next stage the 8 up rows of the same features) times one k phase
// (2048 k-elements when M <= 8, else 1024), i.e. one bulk copy of up to 4 KB per row: the copy
// engine spends a fixed time per copy, and only copies of 2-4 KB and more keep HBM saturated.
// The stages are visited superchunk (<= 256 accumulator rows) -> phase -> row group, in the same
// order by the producer warp (which issues the copies) and the consumers.
//
// Consumers take the stages two at a time: one MMA m16n8k16 computes D[weight row, activation
// column] with the 16 weight rows of a stage pair as the A operand (ldmatrix straight from the
// ring) and the activations as the 8-column B operand.  The activations keep fp32 accuracy by a
// split x * gain = hi + lo into two bf16 parts:
//   V = 4  (M <= 4):  columns 0-3 carry hi, columns 4-7 lo of rows 0-3: one MMA per k16-step;
//   V = 8  (M <= 8):  hi and lo are two MMAs;
//   V = 16 (M <= 16): two column tiles, hi and lo: four MMAs.
// Each of the 8 warps owns a fixed slice of the phase's k range; its B fragments are loaded once
// per phase from the packed activation rows in global memory (L2) and stay in registers for every
// row group, so the steady state touches shared memory only for the weights.  After a stage pair the 8 partial sums of each (weight row,
// activation row) are added in warp order into the per-row accumulators in shared memory.
template <int V> struct LinGeom {
    static constexpr int NS = V == 16 ? 8 : 16;           // k16-steps per warp and stage
    static constexpr int PLEN = NS * 16 * NWARPS;         // k-elements per phase: 2048 or 1024
    static constexpr int FR = V == 4 ? 2 : (V == 8 ? 4 : 8);   // B fragment registers per step
    static constexpr int NACC = V == 16 ? 2 : 1;          // column tiles
};
constexpr int MP = 16;                                    // accumulator columns (activation rows, padded)

struct LinPlan {
    int u0, u1;          // this CTA's units
    int sc_units;        // units per superchunk
    int plen, nph;       // k phases
};

__device__ __forceinline__ LinPlan make_plan(const LinArgs& a, int cta, int nctas) {
    LinPlan p;
    p.u0 = (int)((unsigned)a.N * (unsigned)cta / (unsigned)nctas);          // N * nctas < 2^32 (checked on the host)
    p.u1 = (int)((unsigned)a.N * (unsigned)(cta + 1) / (unsigned)nctas);
    p.sc_units = a.W2 ? SC_ROWS / 2 : SC_ROWS;
    p.plen = a.M <= 8 ? LinGeom<8>::PLEN : LinGeom<16>::PLEN;
    p.nph = (a.K + p.plen - 1) / p.plen;
    return p;
}

// Producer warp: issue the bulk copies of every stage of this operator.
__device__ __noinline__ bool lin_produce(const LinArgs& a, Ctx& c) {
    const int lane = threadIdx.x & 31;
    const LinPlan pl = make_plan(a, c.cta, c.nctas);
    const bool dual = a.W2 != nullptr;
    const __nv_bfloat16* W = reinterpret_cast<const __nv_bfloat16*>(a.W);
    const __nv_bfloat16* W2 = reinterpret_cast<const __nv_bfloat16*>(a.W2);
    char* ring = c.smem + RING_OFF;
    Ctrl* ctl = c.ctl;
    int slot = c.slot; unsigned phase = c.phase; unsigned issued = c.issued;     // ring cursor, kept in registers here
    const unsigned long long policy = l2_evict_first();
    for (int sc0 = pl.u0; sc0 < pl.u1; sc0 += pl.sc_units) {
        const int sc1 = min(pl.u1, sc0 + pl.sc_units);
        const int ngrp = (sc1 - sc0 + ST_ROWS - 1) / ST_ROWS;
        const int nst = dual ? 2 * ngrp : ngrp;
        for (int ph = 0; ph < pl.nph; ++ph) {
            const int p0 = ph * pl.plen, len = min(pl.plen, a.K - p0);
            for (int si = 0; si < nst; ++si) {
                const int base = sc0 + (dual ? si >> 1 : si) * ST_ROWS;
                const int nvalid = min(ST_ROWS, sc1 - base);
                const __nv_bfloat16* src = ((dual && (si & 1)) ? W2 : W) + (size_t)(base + lane) * a.K + p0;
                int ok = 1;
                if (lane == 0) ok = mbar_wait(c, &ctl->empty[slot], phase ^ 1u, 40) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { c.slot = slot; c.phase = phase; c.issued = issued; return false; }
                if (lane == 0) mbar_arrive_expect_tx(&ctl->full[slot], (unsigned)(nvalid * len * 2));
                __syncwarp();
                if (lane < nvalid) bulk_g2s(ring + (size_t)slot * SLOT_BYTES + lane * ST_ROW_BYTES, src, (unsigned)(len * 2), &ctl->full[slot], policy);
                issued++;
                if (++slot == RING) { slot = 0; phase ^= 1u; }
            }
        }
    }
    c.slot = slot; c.phase = phase; c.issued = issued;
    return true;
}

// Producer warp, after a failed wait: let the copies it still has in flight land before the CTA exits.
__device__ void ring_drain(Ctx& c) {
    if ((threadIdx.x & 31) != 0) return;
    const unsigned n = c.issued < (unsigned)RING ? c.issued : (unsigned)RING;
    int s = c.slot; unsigned ph = c.phase;
    for (unsigned i = 0; i < n; ++i) {
        if (--s < 0) { s = RING - 1; ph ^= 1u; }
        const long long t0 = clock64();
        while (!mbar_try_wait(&c.ctl->full[s], ph)) {
            if ((unsigned long long)(clock64() - t0) > c.wait_clk) break;
        }
    }
}

__device__ __forceinline__ void split_hi_lo(float2 v, unsigned& hi, unsigned& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(v.x, v.y);
    const float2 f = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(v.x - f.x, v.y - f.y);
    hi = *reinterpret_cast<const unsigned*>(&h);
    lo = *reinterpret_cast<const unsigned*>(&l);
}

// Shared-memory work area of the streamed path (floats, from WORK_OFF).
constexpr int LW_RED = 0;                                 // [2][NWARPS][16][8] partial sums of a stage pair
constexpr int LW_ACC = LW_RED + 2 * NWARPS * 128;         // [SC_ROWS][MP] row accumulators
constexpr int LW_RS = LW_ACC + SC_ROWS * MP;              // [M_MAX] 1/rms of the input rows
constexpr int LW_RSP = LW_RS + M_MAX;                     // [M_MAX][16] partial sums of squares of the input rows
constexpr int LW_SSW = LW_RSP + M_MAX * 16;               // [NWARPS][M_MAX] sums of squares of the output rows
constexpr int PRE_NU = 64;                                // residual / gain values are prefetched for up to this many units
constexpr int LW_PRES = LW_SSW + NWARPS * M_MAX;          // [M_MAX][PRE_NU] residual values
constexpr int LW_PREG = LW_PRES + M_MAX * PRE_NU;         // [2][PRE_NU] gains of the packed outputs
constexpr int LW_END = LW_PREG + 2 * PRE_NU;
static_assert(LW_END * 4 <= WORK_BYTES, "linear work area too large");

__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}

// Epilogue of the streamed path for everything but the LM head: turns the accumulators of nu output
// units x M rows (acc_s, 1/rms in rs) into fp32 rows, packed copies and per-CTA sums of squares.
// Thread (r, m): m = tid mod 2^ceil(log2 M), so that the lanes of a warp that share m can add their
// squares by shuffles in a fixed order.  Every consumer thread calls it; ssq_acc (threads < M)
// accumulates over superchunks.
__device__ __forceinline__ void emit_rows(const LinArgs& a, float* wk, int sc0, int nu, bool prefetched, float& ssq_acc) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = a.M;
    const float* acc_s = wk + LW_ACC;
    const float* rs = wk + LW_RS;
    float* ssw = wk + LW_SSW;
    const int sh = M <= 1 ? 0 : (M <= 2 ? 1 : (M <= 4 ? 2 : (M <= 8 ? 3 : 4)));
    const int mp = 1 << sh;
    const int m = tid & (mp - 1);
    float ssl = 0.f;
    if (m < M) {
        for (int r = tid >> sh; r < nu; r += NTHREADS >> sh) {
            float v;
            if (a.epi == EPI_SWIGLU) {
                const int srow = (r >> 3) * 16 + (r & 7);
                v = silu_f(acc_s[(size_t)srow * MP + m] * rs[m]) * (acc_s[(size_t)(srow + 8) * MP + m] * rs[m]);
            } else {
                v = acc_s[(size_t)r * MP + m] * rs[m];
                if (a.epi == EPI_RESID)
                    v += prefetched ? wk[LW_PRES + m * PRE_NU + r] : ldcg_f(a.resid + (size_t)m * a.ldr + sc0 + r);
            }
            const int row = sc0 + r;
            if (a.out) a.out[(size_t)m * a.ldo + row] = v;
            ssl += v * v;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (a.pk[q].ptr) {
                    float pv = v;
                    if (a.pk[q].gain) pv *= prefetched ? wk[LW_PREG + q * PRE_NU + r] : __ldg(a.pk[q].gain + row);
                    pk_store(a.pk[q].ptr + (size_t)m * a.ldpk_out, row, pv);
                }
            }
        }
    }
    if (a.ssq_out) {
        for (int o = 16; o >= mp; o >>= 1) ssl += __shfl_xor_sync(0xffffffffu, ssl, o);
        if (lane < mp) ssw[warp * M_MAX + lane] = ssl;
        cta_sync();
        if (tid < M) {
            float sres = 0.f;
            for (int w = 0; w < NWARPS; ++w) sres += ssw[w * M_MAX + tid];
            ssq_acc += sres;
        }
    }
}

template <int V>
__device__ __noinline__ void lin_consume(const LinArgs& a, Ctx& c) {
    using G = LinGeom<V>;
    constexpr int NS = G::NS, FR = G::FR, NACC = G::NACC;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int M = a.M, K = a.K;
    const bool dual = a.W2 != nullptr;
    const LinPlan pl = make_plan(a, c.cta, c.nctas);

    float* wk = reinterpret_cast<float*>(c.smem + WORK_OFF);
    float* red = wk + LW_RED;
    float* acc_s = wk + LW_ACC;
    float* rs = wk + LW_RS;
    const char* ring = c.smem + RING_OFF;
    Ctrl* ctl = c.ctl;
    const int nctas = c.nctas, cta = c.cta;
    int slot = c.slot; unsigned phase = c.phase;              // ring cursor, kept in registers here

    HeadStat hs[2];                                                        // EPI_HEAD: this warp tracks rows warp, warp + 8
    hs[0].zmax = hs[1].zmax = 0.f; hs[0].sum = hs[1].sum = 0.f; hs[0].arg = hs[1].arg = 0;
    bool ok = true;
    int buf = 0;
    float ssq_acc = 0.f;

    // ---- fetched early, used in the epilogue: the input rows' sums of squares, residual values, output gains.
    // The requests go out right behind the first phase's fragment loads, which the first MMA waits for.
    const int nu0 = min(pl.u1 - pl.u0, pl.sc_units);
    const bool prefetched = nu0 <= PRE_NU;
    bool pre_pending = true;
    auto epilogue_prefetch = [&]() {
        if (a.ssq_in) {
            // thread (m, j) adds the partial sums of CTAs j, j + 16, ... of row m
            const int m = tid >> 4, j = tid & 15;
            float part = 0.f;
            if (m < M) for (int q = j; q < nctas; q += 16) part += ldcg_f(a.ssq_in + (size_t)m * nctas + q);
            wk[LW_RSP + tid] = part;
        }
        if (prefetched && a.epi != EPI_HEAD) {
            if (a.epi == EPI_RESID)
                for (int i = tid; i < M * nu0; i += NTHREADS) cp_async4(wk + LW_PRES + (i / nu0) * PRE_NU + i % nu0, a.resid + (size_t)(i / nu0) * a.ldr + pl.u0 + i % nu0);
#pragma unroll
            for (int q = 0; q < 2; ++q)
                if (a.pk[q].ptr && a.pk[q].gain)
                    for (int i = tid; i < nu0; i += NTHREADS) cp_async4(wk + LW_PREG + q * PRE_NU + i, a.pk[q].gain + pl.u0 + i);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // this lane's rows of the packed input: V = 4: row g & 3 (hi for g < 4, lo for g >= 4); else rows g (and g + 8)
    const int xrow = V == 4 ? (g & 3) : g;
    const unsigned char* xlane = a.xpk + (size_t)xrow * a.ldpk + (size_t)warp * NS * 64 + t * 16 + (V == 4 ? (g >> 2) * 8 : 0);

    for (int sc0 = pl.u0; sc0 < pl.u1; sc0 += pl.sc_units) {
        const int sc1 = min(pl.u1, sc0 + pl.sc_units);
        const int nu = sc1 - sc0;
        const int ngrp = (nu + ST_ROWS - 1) / ST_ROWS;
        const int nst = dual ? 2 * ngrp : ngrp;
        for (int ph = 0; ph < pl.nph; ++ph) {
            const int p0 = ph * pl.plen, len = min(pl.plen, K - p0);
            const int nsteps = len / 16;
            // ---- B fragments of this warp's k slice, kept in registers for every row group of the phase
            // (every load is issued before any is used: steps past the end of the phase and rows >= M re-read valid
            // data and are zeroed afterwards)
            unsigned fr[NS][FR];
            {
                const int last = nsteps - 1 - warp * NS;         // last valid step of this warp (< 0: none)
                const unsigned char* pbase = xlane + (size_t)(p0 / 16) * 64;
#pragma unroll
                for (int s = 0; s < NS; ++s) {
                    const unsigned char* px = pbase + (size_t)max(min(s, last), -warp * NS) * 64;
                    if (V == 4) {
                        const uint2 v = __ldcg(reinterpret_cast<const uint2*>(xrow < M ? px : px - (size_t)xrow * a.ldpk));
                        fr[s][0] = v.x; fr[s][1] = v.y;
                    } else {
#pragma unroll
                        for (int n = 0; n < NACC; ++n) {
                            const int row = xrow + 8 * n;
                            const uint4 v = __ldcg(reinterpret_cast<const uint4*>(row < M ? px + (size_t)(8 * n) * a.ldpk : px - (size_t)xrow * a.ldpk));
                            fr[s][4 * n + 0] = v.x; fr[s][4 * n + 1] = v.y; fr[s][4 * n + 2] = v.z; fr[s][4 * n + 3] = v.w;
                        }
                    }
                }
                if (pre_pending) { pre_pending = false; epilogue_prefetch(); }
#pragma unroll
                for (int s = 0; s < NS; ++s) {
                    const bool sv = s <= last;
                    if (V == 4) {
                        if (!(sv && xrow < M)) { fr[s][0] = 0u; fr[s][1] = 0u; }
                    } else {
#pragma unroll
                        for (int n = 0; n < NACC; ++n)
                            if (!(sv && xrow + 8 * n < M)) { fr[s][4 * n + 0] = 0u; fr[s][4 * n + 1] = 0u; fr[s][4 * n + 2] = 0u; fr[s][4 * n + 3] = 0u; }
                    }
                }
            }
            // ---- the row groups of this phase, two stages (16 weight rows) at a time
            const uint32_t a_lane = (uint32_t)((lane & 7) * ST_ROW_BYTES + (warp * NS * 16 + (lane >> 4) * 8) * 2);
            for (int si = 0; si < nst; si += 2) {
                const bool two = si + 1 < nst;
                const int slot_a = slot;
                const int slot_b = two ? (slot_a + 1 == RING ? 0 : slot_a + 1) : slot_a;
                const unsigned phase_b = (two && slot_a + 1 == RING) ? phase ^ 1u : phase;
                float acc[4][4];
#pragma unroll
                for (int q = 0; q < 4; ++q) { acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.f; }
                if (ok) ok = mbar_wait(c, &ctl->full[slot_a], phase, 41);
                if (ok && two) ok = mbar_wait(c, &ctl->full[slot_b], phase_b, 41);
                if (ok) {
                    // ldmatrix x4: matrices 0, 2 = rows 0-7 (first stage), 1, 3 = rows 8-15 (second stage); k halves 0-7 | 8-15
                    const uint32_t a_base = smem_u32(ring + (size_t)((lane & 8) ? slot_b : slot_a) * SLOT_BYTES) + a_lane;
                    // the weight fragments are fetched PD steps ahead of the MMA that uses them (the loads and the MMAs
                    // issue in program order, so a load right before its MMA would expose its latency at every step);
                    // loads past the phase's last step stay inside the slot and are never used
                    constexpr int PD = V == 4 ? 4 : 2;
                    unsigned af[PD][4];
#pragma unroll
                    for (int s = 0; s < PD; ++s) ldmatrix_x4(af[s], a_base + (uint32_t)s * 32u);
#pragma unroll
                    for (int s = 0; s < NS; ++s) {
                        if (warp * NS + s < nsteps) {
                            if (V == 4) {
                                mma_bf16_16816(acc[s & 3], af[s % PD], fr[s][0], fr[s][1]);
                            } else if (V == 8) {
                                mma_bf16_16816(acc[(s & 1) * 2], af[s % PD], fr[s][0], fr[s][1]);
                                mma_bf16_16816(acc[(s & 1) * 2 + 1], af[s % PD], fr[s][2], fr[s][3]);
                            } else {
                                mma_bf16_16816(acc[0], af[s % PD], fr[s][0], fr[s][1]);
                                mma_bf16_16816(acc[1], af[s % PD], fr[s][2], fr[s][3]);
                                mma_bf16_16816(acc[2], af[s % PD], fr[s][FR - 4], fr[s][FR - 3]);
                                mma_bf16_16816(acc[3], af[s % PD], fr[s][FR - 2], fr[s][FR - 1]);
                            }
                        }
                        if (s + PD < NS) ldmatrix_x4(af[s % PD], a_base + (uint32_t)(s + PD) * 32u);
                    }
                }
                __syncwarp();
                if (ok && lane == 0) { mbar_arrive(&ctl->empty[slot_a]); if (two) mbar_arrive(&ctl->empty[slot_b]); }
                slot = slot_b; phase = phase_b;
                if (++slot == RING) { slot = 0; phase ^= 1u; }
                // ---- add the k-slices in warp order into the row accumulators
                if (V == 16) cta_sync();                     // single partial-sum buffer: the previous pair's sums have been read
                float* r = red + (size_t)(V == 16 ? 0 : buf) * NWARPS * 128 + (size_t)warp * NACC * 128;
                if (V == 16) {
                    // acc[0] / acc[1]: hi / lo of columns 0-7; acc[2] / acc[3]: hi / lo of columns 8-15
                    *reinterpret_cast<float2*>(r + g * 8 + 2 * t) = make_float2(acc[0][0] + acc[1][0], acc[0][1] + acc[1][1]);
                    *reinterpret_cast<float2*>(r + (g + 8) * 8 + 2 * t) = make_float2(acc[0][2] + acc[1][2], acc[0][3] + acc[1][3]);
                    *reinterpret_cast<float2*>(r + 128 + g * 8 + 2 * t) = make_float2(acc[2][0] + acc[3][0], acc[2][1] + acc[3][1]);
                    *reinterpret_cast<float2*>(r + 128 + (g + 8) * 8 + 2 * t) = make_float2(acc[2][2] + acc[3][2], acc[2][3] + acc[3][3]);
                } else {
                    *reinterpret_cast<float2*>(r + g * 8 + 2 * t) =
                        make_float2((acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]), (acc[0][1] + acc[1][1]) + (acc[2][1] + acc[3][1]));
                    *reinterpret_cast<float2*>(r + (g + 8) * 8 + 2 * t) =
                        make_float2((acc[0][2] + acc[1][2]) + (acc[2][2] + acc[3][2]), (acc[0][3] + acc[1][3]) + (acc[2][3] + acc[3][3]));
                }
                cta_sync();
                {
                    // element (weight row r16, activation row m) of the pair; for M <= 8 every thread adds a share of the
                    // eight k-slices and a fixed butterfly joins the shares, so that no warp lags behind the others
                    if (V == 16) {
                        const int r16 = tid >> 4, m = tid & 15;
                        const float* rb = red + (m >> 3) * 128 + r16 * 8 + (m & 7);
                        float v = 0.f;
#pragma unroll
                        for (int w = 0; w < NWARPS; ++w) v += rb[w * NACC * 128];
                        float* dst = acc_s + (size_t)((si >> 1) * 16 + r16) * MP + m;
                        *dst = ph == 0 ? v : *dst + v;
                    } else {
                        constexpr int TPE = V == 4 ? 4 : 2;                  // threads per element
                        constexpr int WPT = NWARPS / TPE;                    // k-slices per thread
                        const int e = tid / TPE, q = tid % TPE;
                        const int r16 = V == 4 ? e >> 2 : e >> 3;
                        const int m = V == 4 ? e & 3 : e & 7;
                        const float* rb = red + (size_t)buf * NWARPS * 128 + r16 * 8 + m;
                        float v = 0.f;
#pragma unroll
                        for (int w = 0; w < WPT; ++w) v += V == 4 ? rb[(q * WPT + w) * 128] + rb[(q * WPT + w) * 128 + 4] : rb[(q * WPT + w) * 128];
#pragma unroll
                        for (int o = 1; o < TPE; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                        if (q == 0) {
                            float* dst = acc_s + (size_t)((si >> 1) * 16 + r16) * MP + m;
                            *dst = ph == 0 ? v : *dst + v;
                        }
                    }
                }
                buf ^= 1;
            }
        }
        // ---- epilogue of this superchunk
        if (sc0 == pl.u0) {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            cta_sync();
            if (tid < M_MAX) {
                float r = 1.0f;
                if (a.ssq_in && tid < M) {
                    float ss = 0.f;
                    for (int j = 0; j < 16; ++j) ss += wk[LW_RSP + tid * 16 + j];
                    r = rsqrtf(ss / (float)K + a.eps);
                }
                rs[tid] = r;
            }
        }
        cta_sync();
        if (a.epi == EPI_HEAD) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int m = warp + q * NWARPS;
                if (m < M) {
                    const float f = rs[m] * a.scale;
                    float zm = -INFINITY; int im = 0x7fffffff;
                    for (int r = lane; r < nu; r += 32) {
                        const float z = acc_s[(size_t)r * MP + m] * f;
                        if (a.logits_dbg) a.logits_dbg[(size_t)m * a.ld_dbg + sc0 + r] = z;
                        if (arg_better(z, sc0 + r, zm, im)) { zm = z; im = sc0 + r; }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const float z2 = __shfl_xor_sync(0xffffffffu, zm, o);
                        const int i2 = __shfl_xor_sync(0xffffffffu, im, o);
                        if (arg_better(z2, i2, zm, im)) { zm = z2; im = i2; }
                    }
                    float e = 0.f;
                    for (int r = lane; r < nu; r += 32) e += expf(acc_s[(size_t)r * MP + m] * f - zm);
                    e = warp_sum(e);
                    if (nu > 0) head_merge(hs[q], zm, e, im);
                }
            }
        } else {
            emit_rows(a, wk, sc0, nu, prefetched && sc0 == pl.u0, ssq_acc);
        }
        cta_sync();                                  // acc_s is rewritten by the next superchunk / operator
    }
    if (a.epi == EPI_HEAD && lane == 0) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int m = warp + q * NWARPS;
            if (m < M) a.head_part[(size_t)cta * M_MAX + m] = make_float4(hs[q].zmax, hs[q].sum, __int_as_float(hs[q].arg), 0.f);
        }
    }
    if (a.epi != EPI_HEAD && a.ssq_out && tid < M) a.ssq_out[(size_t)tid * nctas + cta] = ssq_acc;
    c.slot = slot; c.phase = phase;
}

// Rows that do not come out of a linear operator (token embeddings): every CTA takes its slice of
// the d columns, places the values where the epilogue expects accumulators and emits them like
// an operator output (fp32 rows, packed copies, sums of squares).  value(m, e) is given by the caller.
template <typename F>
__device__ __forceinline__ void emit_plain_rows(LinArgs& a, Ctx& c, F value) {
    const int tid = threadIdx.x;
    float* wk = reinterpret_cast<float*>(c.smem + WORK_OFF);
    const int u0 = (int)((unsigned)a.N * (unsigned)c.cta / (unsigned)c.nctas);
    const int u1 = (int)((unsigned)a.N * (unsigned)(c.cta + 1) / (unsigned)c.nctas);
    float ssq_acc = 0.f;
    a.epi = EPI_STORE;
    if (tid < M_MAX) wk[LW_RS + tid] = 1.0f;
    for (int sc0 = u0; sc0 < u1; sc0 += SC_ROWS) {
        const int nu = min(SC_ROWS, u1 - sc0);
        for (int idx = tid; idx < nu * a.M; idx += NTHREADS) {
            const int r = idx % nu, m = idx / nu;
            wk[LW_ACC + (size_t)r * MP + m] = value(m, sc0 + r);
        }
        cta_sync();
        emit_rows(a, wk, sc0, nu, false, ssq_acc);
        cta_sync();
    }
    if (a.ssq_out && tid < a.M) a.ssq_out[(size_t)tid * c.nctas + c.cta] = ssq_acc;
}

// Plain path for any storage type (fp32 models, odd shapes, and a cross-check of the tensor-core
// path): activations staged in shared memory as fp32, one output row per warp at a time.
template <typename WT>
__device__ __noinline__ void lin_simple(const LinArgs& a, Ctx& c) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int M = a.M, K = a.K;
    const WT* W = reinterpret_cast<const WT*>(a.W);
    const WT* W2 = reinterpret_cast<const WT*>(a.W2);
    const bool dual = W2 != nullptr;
    char* work = c.smem + RING_OFF;
    float* xs = reinterpret_cast<float*>(work);                          // [M][K]
    float* rs = reinterpret_cast<float*>(work + SIMPLE_XS_BYTES);        // [M_MAX]
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
    cta_sync();

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
        cta_sync();
        if (tid < M) {
            HeadStat tot; tot.zmax = 0.f; tot.sum = 0.f; tot.arg = 0;
            for (int w = 0; w < NWARPS; ++w)
                head_merge(tot, wst[(w * M_MAX + tid) * 3 + 0], wst[(w * M_MAX + tid) * 3 + 1],
                           __float_as_int(wst[(w * M_MAX + tid) * 3 + 2]));
            a.head_part[(size_t)c.cta * M_MAX + tid] = make_float4(tot.zmax, tot.sum, __int_as_float(tot.arg), 0.f);
        }
    }
    cta_sync();
}

// One linear operator, called by every thread of the CTA; `stream` selects the streamed tensor-core
// path (bf16 weights, every K a multiple of 16; decided once per model so that the packed activation
// rows exist wherever they are read).  Consumers return after their part; whether the grid must stop
// is learnt at the next grid barrier.  The producer returns false when one of its waits gave up.
template <typename WT>
__device__ __forceinline__ bool linear_consumer(const LinArgs* sa, Ctx& c, bool stream, bool publish) {
    if (publish) cta_sync();
    if (stream) {
        if (sa->M <= 4) lin_consume<4>(*sa, c); else if (sa->M <= 8) lin_consume<8>(*sa, c); else lin_consume<16>(*sa, c);
    } else {
        lin_simple<WT>(*sa, c);
    }
    return true;
}
__device__ __forceinline__ bool linear_producer(const LinArgs* sa, Ctx& c, bool stream, bool publish) {
    if (!stream) return true;
    if (publish) __syncwarp();
    return lin_produce(*sa, c);
}
template <typename WT>
__device__ __forceinline__ bool linear_op(const LinArgs* sa, Ctx& c, bool stream, bool publish) {
    // sa points into this role's operator table in shared memory; publish: the table was written just before
    return c.producer ? linear_producer(sa, c, stream, publish) : linear_consumer<WT>(sa, c, stream, publish);
}

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

// The same merge by a whole warp: every lane merges the partials of CTAs lane, lane + 32, ... (independent loads, one
// round trip instead of one per CTA), then a butterfly of merges leaves the identical total in every lane (the merge
// of two partials is the same whichever of the two lanes computes it).
__device__ __forceinline__ void head_final_warp(const float4* part, int nctas, int m, int& tok, float& p) {
    const int lane = threadIdx.x & 31;
    HeadStat tot; tot.zmax = 0.f; tot.sum = 0.f; tot.arg = 0;
    for (int cta = lane; cta < nctas; cta += 32) {
        const float4 v = __ldcg(part + (size_t)cta * M_MAX + m);
        head_merge(tot, v.x, v.y, __float_as_int(v.z));
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float z = __shfl_xor_sync(0xffffffffu, tot.zmax, o);
        const float sm = __shfl_xor_sync(0xffffffffu, tot.sum, o);
        const int ar = __shfl_xor_sync(0xffffffffu, tot.arg, o);
        head_merge(tot, z, sm, ar);
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
    unsigned char* opk;    // packed copy of out for the output projection (nullable); d * 4 bytes per row
};

// The operators of one layer (or of the adapter / the LM head), prepared together.
struct OpTable { LinArgs lin[4]; AttArgs att; };
static_assert(sizeof(OpTable) <= OP_TABLE_BYTES, "operator table too large");

// Consumer threads only.  One work item = (head, KV split); the eight warps of the CTA cut the item's
// key range into eight slices and run an online-softmax pass over their slice without any CTA
// barrier: a lane owns hd/32 consecutive dimensions, so a key or value row is one coalesced load of
// the warp, q . k is finished by a butterfly of shuffles, and o += p v stays in the lane.  Keys are
// taken eight at a time (their loads are issued together).  The rows of this pass are rotated
// (RoPE), rounded to the cache's storage type and appended to the cache by the item whose key range
// contains them, then read back like any other key.  The warps' (max, sum, o) are merged through
// shared memory; with more than one split every item writes a partial and the last split of a head
// to arrive merges them in split order.
template <typename WT, int DPL> struct AttLoad;          // raw bits of DPL consecutive elements, and their conversion
template <> struct AttLoad<__nv_bfloat16, 4> {
    typedef uint2 Raw;
    static __device__ __forceinline__ Raw ld(const __nv_bfloat16* p) { return __ldcg(reinterpret_cast<const uint2*>(p)); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[4]) {
        v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xffff0000u);
        v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xffff0000u);
    }
};
template <> struct AttLoad<__nv_bfloat16, 2> {
    typedef unsigned Raw;
    static __device__ __forceinline__ Raw ld(const __nv_bfloat16* p) { return __ldcg(reinterpret_cast<const unsigned*>(p)); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[2]) { v[0] = __uint_as_float(r << 16); v[1] = __uint_as_float(r & 0xffff0000u); }
};
template <> struct AttLoad<__nv_bfloat16, 1> {
    typedef unsigned short Raw;
    static __device__ __forceinline__ Raw ld(const __nv_bfloat16* p) { return __ldcg(reinterpret_cast<const unsigned short*>(p)); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[1]) { v[0] = __uint_as_float((unsigned)r << 16); }
};
template <> struct AttLoad<float, 4> {
    typedef float4 Raw;
    static __device__ __forceinline__ Raw ld(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[4]) { v[0] = r.x; v[1] = r.y; v[2] = r.z; v[3] = r.w; }
};
template <> struct AttLoad<float, 2> {
    typedef float2 Raw;
    static __device__ __forceinline__ Raw ld(const float* p) { return __ldcg(reinterpret_cast<const float2*>(p)); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[2]) { v[0] = r.x; v[1] = r.y; }
};
template <> struct AttLoad<float, 1> {
    typedef float Raw;
    static __device__ __forceinline__ Raw ld(const float* p) { return __ldcg(p); }
    static __device__ __forceinline__ void cvt(const Raw& r, float (&v)[1]) { v[0] = r; }
};

constexpr int ATT_G = 8;           // keys per group
constexpr int ATT_RB = 4;          // rows per block
constexpr int ATT_MB_STRIDE = HD_MAX + 2;   // merge buffer row: o[hd], max, sum

__device__ __forceinline__ float ex2f(float x) {             // 2^x, one special-function instruction
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One warp: rows i0 .. i0+nr-1 of the pass against keys [kb, ke) of head hh.  Scores are kept in the log2
// domain (q is pre-scaled by log2(e) / sqrt(hd)), so every exponential is one ex2.  The loads of the next
// key group are in flight while the current one is reduced.  A group's 8 x 4 partial dot products are summed
// by a transposing butterfly (31 shuffles) that leaves score (key j, row r) in lane 4 j + r; that lane does the
// online-softmax update of its row (lanes sharing r hold the same running max and sum), and the 32 probabilities
// reach every lane through a few words of shared memory for o += p v.
template <typename WT, int DPL>
__device__ __forceinline__ void att_warp_slice(const Dev& D, const AttArgs& a, int hh, int i0, int nr, int kb, int ke,
                                               const float* qs, float* pbuf, float& m_lane, float& l_lane, float (&o)[ATT_RB][DPL]) {
    typedef typename AttLoad<WT, DPL>::Raw Raw;
    static_assert(ATT_G == 8 && ATT_RB == 4, "the butterfly below is written for 8 keys x 4 rows");
    const int lane = threadIdx.x & 31;
    const int jl = lane >> 2, rl = lane & 3;
    const int H = D.dm.H, hd = D.dm.hd, psh = D.dm.ps_shift, psm = D.dm.page_size - 1;
    const int pos0 = a.pos0;
    const WT* kc = reinterpret_cast<const WT*>(a.kc);
    const WT* vc = reinterpret_cast<const WT*>(a.vc);
    const int* page_table = D.page_table;
    float q[ATT_RB][DPL];
#pragma unroll
    for (int r = 0; r < ATT_RB; ++r) {
#pragma unroll
        for (int e = 0; e < DPL; ++e) { o[r][e] = 0.f; q[r][e] = r < nr ? qs[(i0 + r) * HD_MAX + lane * DPL + e] : 0.f; }
    }
    m_lane = -INFINITY; l_lane = 0.f;
    if (kb >= ke) return;
    // page table entries of a window of keys live in the lanes (lane p holds page first_page + p)
    const int win = max(ATT_G, ((31 << psh) >> 3) << 3);
    int wstart = kb, first_page = kb >> psh;
    int pgs = __ldg(page_table + min(first_page + lane, D.dm.n_pages - 1));
    Raw kr[ATT_G], vr[ATT_G];
    auto issue = [&](int g0) {
        if (g0 >= wstart + win) { wstart = g0; first_page = g0 >> psh; pgs = __ldg(page_table + min(first_page + lane, D.dm.n_pages - 1)); }
#pragma unroll
        for (int j = 0; j < ATT_G; ++j) {
            const int pos = min(g0 + j, ke - 1);
            const int pg = __shfl_sync(0xffffffffu, pgs, (pos >> psh) - first_page);
            const size_t base = ((((size_t)pg * H + hh) << psh) + (pos & psm)) * hd + lane * DPL;
            kr[j] = AttLoad<WT, DPL>::ld(kc + base);
            vr[j] = AttLoad<WT, DPL>::ld(vc + base);
        }
    };
    issue(kb);
    for (int g0 = kb; g0 < ke; g0 += ATT_G) {
        float kv[ATT_G][DPL], vv[ATT_G][DPL];
#pragma unroll
        for (int j = 0; j < ATT_G; ++j) { AttLoad<WT, DPL>::cvt(kr[j], kv[j]); AttLoad<WT, DPL>::cvt(vr[j], vv[j]); }
        if (g0 + ATT_G < ke) issue(g0 + ATT_G);
        float v[ATT_G * ATT_RB];
#pragma unroll
        for (int j = 0; j < ATT_G; ++j) {
#pragma unroll
            for (int r = 0; r < ATT_RB; ++r) {
                float dsum = 0.f;
#pragma unroll
                for (int e = 0; e < DPL; ++e) dsum = fmaf(q[r][e], kv[j][e], dsum);
                v[j * ATT_RB + r] = dsum;
            }
        }
        // transposing butterfly: after the step with offset `ofs` a lane keeps the half of its values selected by that
        // bit of its lane index, summed with the partner's; in the end lane L holds the full sum of value L
#pragma unroll
        for (int ofs = 16; ofs > 0; ofs >>= 1) {
            const bool up = (lane & ofs) != 0;
#pragma unroll
            for (int i = 0; i < ofs; ++i) {
                const float send = up ? v[i] : v[i + ofs];
                const float keep = up ? v[i + ofs] : v[i];
                v[i] = keep + __shfl_xor_sync(0xffffffffu, send, ofs);
            }
        }
        const int pos = g0 + jl;
        float sv = (pos < ke && rl < nr && pos <= pos0 + i0 + rl) ? v[0] : -INFINITY;
        float mg = sv;
        mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, 4));
        mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, 8));
        mg = fmaxf(mg, __shfl_xor_sync(0xffffffffu, mg, 16));
        const float mn = fmaxf(m_lane, mg);
        const float p = (sv == -INFINITY) ? 0.f : ex2f(sv - mn);
        const float cf = (m_lane == -INFINITY) ? 0.f : ex2f(m_lane - mn);
        float psum = p;
        psum += __shfl_xor_sync(0xffffffffu, psum, 4);
        psum += __shfl_xor_sync(0xffffffffu, psum, 8);
        psum += __shfl_xor_sync(0xffffffffu, psum, 16);
        l_lane = l_lane * cf + psum;
        m_lane = mn;
        __syncwarp();
        pbuf[lane] = p;
        if (jl == 0) pbuf[32 + rl] = cf;
        __syncwarp();
        const float4 cfv = *reinterpret_cast<const float4*>(pbuf + 32);
        const float cfa[4] = {cfv.x, cfv.y, cfv.z, cfv.w};
#pragma unroll
        for (int r = 0; r < ATT_RB; ++r) {
#pragma unroll
            for (int e = 0; e < DPL; ++e) o[r][e] *= cfa[r];
        }
#pragma unroll
        for (int j = 0; j < ATT_G; ++j) {
            const float4 pj = *reinterpret_cast<const float4*>(pbuf + j * 4);
            const float pa[4] = {pj.x, pj.y, pj.z, pj.w};
#pragma unroll
            for (int r = 0; r < ATT_RB; ++r) {
#pragma unroll
                for (int e = 0; e < DPL; ++e) o[r][e] = fmaf(pa[r], vv[j][e], o[r][e]);
            }
        }
    }
}

// The last split of a head to arrive merges the S partial (max, sum, o) of every row in split order.  SC >= S is the
// compile-time bound of the split loop; U elements per thread are handled together, and every load of such a batch is
// issued before any is used, so that a batch costs one L2 round trip.
template <int SC, int U>
__device__ __forceinline__ void att_merge_splits(const Dev& D, const AttArgs& a, int hh, int S, int M) {
    const int tid = threadIdx.x, H = D.dm.H, hd = D.dm.hd, d = D.dm.d;
    const int total = M * hd;
    for (int idx0 = tid; idx0 < total; idx0 += NTHREADS * U) {
        float2 mlv[U][SC];
        float pov[U][SC];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = idx0 + u * NTHREADS < total ? idx0 + u * NTHREADS : idx0;
            const int i = idx / hd, e = idx % hd;
            const float2* ml = reinterpret_cast<const float2*>(D.att_ml + ((size_t)i * H + hh) * S_CAP * 2);
            const float* po = D.att_po + ((size_t)i * H + hh) * S_CAP * hd + e;
#pragma unroll
            for (int q = 0; q < SC; ++q) {
                const int qq = q < S ? q : 0;
                mlv[u][q] = __ldcg(ml + qq);
                pov[u][q] = ldcg_f(po + (size_t)qq * hd);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = idx0 + u * NTHREADS;
            if (idx < total) {
                const int i = idx / hd, e = idx % hd;
                float mx = -INFINITY;
#pragma unroll
                for (int q = 0; q < SC; ++q) if (q < S) mx = fmaxf(mx, mlv[u][q].x);
                float den = 0.f, num = 0.f;
#pragma unroll
                for (int q = 0; q < SC; ++q) {
                    if (q < S && mlv[u][q].x != -INFINITY) {
                        const float w = ex2f(mlv[u][q].x - mx);
                        den += mlv[u][q].y * w;
                        num += pov[u][q] * w;
                    }
                }
                const float ov = num / den;
                a.out[(size_t)i * d + hh * hd + e] = ov;
                if (a.opk) pk_store(a.opk + (size_t)i * d * 4, hh * hd + e, ov);
            }
        }
    }
}

template <typename WT, int DPL>
__device__ __noinline__ void attention_impl(const Dev& D, const AttArgs& a, Ctx& c) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int H = D.dm.H, hd = D.dm.hd, d = D.dm.d, ps = D.dm.page_size;
    const int M = a.M, pos0 = a.pos0;
    const int T = pos0 + M;
    const int half = hd >> 1;
    // number of KV splits: the one that leaves the fewest keys on the busiest CTA
    int S = 1;
    {
        const float inv_ctas = 1.0f / (float)c.nctas;
        float best = -1.f;
#pragma unroll
        for (int sc = 1; sc <= S_CAP; ++sc) {
            const int chunk_ = (T + sc - 1) / sc;                                   // sc is a constant after unrolling
            const float waves = ceilf((float)(H * sc) * inv_ctas - 1e-4f);
            const float cost = waves * (float)(chunk_ + 48);                        // + a fixed cost per item
            if ((sc == 1 || chunk_ >= 32) && (best < 0.f || cost < best)) { best = cost; S = sc; }
        }
    }
    const int chunk = (T + S - 1) / S;
    const float sc = rsqrtf((float)hd) * 1.4426950408889634f;      // 1/sqrt(hd), and log2(e): scores live in the log2 domain
    WT* kc = reinterpret_cast<WT*>(a.kc);
    WT* vc = reinterpret_cast<WT*>(a.vc);

    float* qs = reinterpret_cast<float*>(c.smem + WORK_OFF);       // [M_MAX][HD_MAX]
    float* mb = qs + M_MAX * HD_MAX;                               // [NWARPS][ATT_RB][ATT_MB_STRIDE]
    float* pbuf = mb + NWARPS * ATT_RB * ATT_MB_STRIDE + warp * 40;      // [NWARPS][40] probabilities of a key group

    for (int item = c.cta; item < H * S; item += c.nctas) {
        const int hh = item / S, s = item % S;
        const int kb = s * chunk, ke = min(T, kb + chunk);
        // q rows: RoPE, pre-scaled by 1/sqrt(hd) (loads first: the angle arithmetic runs while they are in flight)
        for (int idx = tid; idx < M * half; idx += NTHREADS) {
            const int i = idx / half, e = idx % half;
            const float x1 = ldcg_f(a.qkv + (size_t)i * 3 * d + hh * hd + e);
            const float x2 = ldcg_f(a.qkv + (size_t)i * 3 * d + hh * hd + e + half);
            float cs, sn; rope_cs(D, pos0 + i, e, cs, sn);
            qs[i * HD_MAX + e] = (x1 * cs - x2 * sn) * sc;
            qs[i * HD_MAX + e + half] = (x2 * cs + x1 * sn) * sc;
        }
        // append this pass's K / V rows that fall into my key range (every load of an element before its first use)
        {
            const int nb = max(kb, pos0), ne = ke;
            for (int idx = tid; idx < (ne - nb) * half; idx += NTHREADS) {
                const int pos = nb + idx / half, e = idx % half, i = pos - pos0;
                const float* src = a.qkv + (size_t)i * 3 * d + hh * hd;
                const float k1 = ldcg_f(src + d + e), k2 = ldcg_f(src + d + e + half);
                const float v1 = ldcg_f(src + 2 * d + e), v2 = ldcg_f(src + 2 * d + e + half);
                const int page = __ldg(D.page_table + (pos >> D.dm.ps_shift));
                float cs, sn; rope_cs(D, pos, e, cs, sn);
                const size_t base = (((size_t)page * H + hh) * ps + (pos & (ps - 1))) * hd;
                kc[base + e] = float_to_wt<WT>(k1 * cs - k2 * sn);
                kc[base + e + half] = float_to_wt<WT>(k2 * cs + k1 * sn);
                vc[base + e] = float_to_wt<WT>(v1);
                vc[base + e + half] = float_to_wt<WT>(v2);
            }
        }
        cta_sync();
        // this warp's slice of the item's keys, in whole groups
        const int nkeys = ke - kb;
        const int per = ((nkeys + NWARPS - 1) / NWARPS + ATT_G - 1) / ATT_G * ATT_G;
        const int wb = min(ke, kb + warp * per), we = min(ke, wb + per);
        for (int i0 = 0; i0 < M; i0 += ATT_RB) {
            const int nr = min(ATT_RB, M - i0);
            float m_lane, l_lane, o[ATT_RB][DPL];
            att_warp_slice<WT, DPL>(D, a, hh, i0, nr, wb, we, qs, pbuf, m_lane, l_lane, o);
#pragma unroll
            for (int r = 0; r < ATT_RB; ++r) {
                float* row = mb + ((size_t)warp * ATT_RB + r) * ATT_MB_STRIDE;
#pragma unroll
                for (int e = 0; e < DPL; ++e) row[lane * DPL + e] = o[r][e];
                if (lane == r) { row[HD_MAX] = m_lane; row[HD_MAX + 1] = l_lane; }       // lane r tracks row r
            }
            cta_sync();
            for (int idx = tid; idx < nr * hd; idx += NTHREADS) {
                const int r = idx / hd, e = idx % hd, i = i0 + r;
                float mx = -INFINITY;
#pragma unroll
                for (int w = 0; w < NWARPS; ++w) mx = fmaxf(mx, mb[((size_t)w * ATT_RB + r) * ATT_MB_STRIDE + HD_MAX]);
                float den = 0.f, num = 0.f;
#pragma unroll
                for (int w = 0; w < NWARPS; ++w) {
                    const float* row = mb + ((size_t)w * ATT_RB + r) * ATT_MB_STRIDE;
                    const float mw = row[HD_MAX];
                    if (mw != -INFINITY) {
                        const float wgt = ex2f(mw - mx);
                        den += row[HD_MAX + 1] * wgt;
                        num += row[e] * wgt;
                    }
                }
                if (S == 1) {
                    const float ov = num / den;
                    a.out[(size_t)i * d + hh * hd + e] = ov;
                    if (a.opk) pk_store(a.opk + (size_t)i * d * 4, hh * hd + e, ov);
                } else {
                    D.att_po[(((size_t)i * H + hh) * S_CAP + s) * hd + e] = num;
                    if (e == 0) {
                        D.att_ml[(((size_t)i * H + hh) * S_CAP + s) * 2 + 0] = mx;
                        D.att_ml[(((size_t)i * H + hh) * S_CAP + s) * 2 + 1] = den;
                    }
                }
            }
            cta_sync();
        }
        if (S > 1) {
            __threadfence();
            cta_sync();
            if (tid == 0) {
                const unsigned prev = atomicAdd(D.att_cnt + hh, 1u);
                const int last = (prev == (unsigned)(S - 1));
                c.ctl->att_last = last;
                if (last) { D.att_cnt[hh] = 0u; __threadfence(); }
            }
            cta_sync();
            if (*(volatile int*)&c.ctl->att_last) {
                if (S <= 4) att_merge_splits<4, 4>(D, a, hh, S, M);
                else if (S <= 8) att_merge_splits<8, 2>(D, a, hh, S, M);
                else att_merge_splits<S_CAP, 1>(D, a, hh, S, M);
            }
            cta_sync();
        }
    }
}


// ---- tensor-core attention (bf16 cache, head_dim 64 or 128) ----------------------------------------------------
//
// One pass over the keys for all rows of the pass.  The unit of work is a tile of 16 keys and one group of 8 rows
// (with more than 8 rows, two units take the same tiles, one row group each: the tile's second reader finds it in
// L2, so K and V still leave HBM once).  A unit is one warp when head_dim is 64; with head_dim 128 it is a pair of
// warps that own 64 dims each, which keeps a warp's share of K, V and the output small enough to hold two tiles in
// registers.  Everything a tile needs travels global memory -> registers -> tensor core:
//   S = K Q^T   m16n8k16, keys on the M side, rows on the N side.  A lane loads 16 bytes (8 dims) of two key rows;
//               which dims sit at which k position of the instruction does not matter for a dot product as long as
//               the Q fragment (read from shared memory, rotated, pre-scaled, split into bf16 hi + lo) uses the same
//               assignment, so no transposition is needed.  The two warps of a pair add their halves of the dot
//               products through shared memory (one named barrier per tile); both then hold the same scores.
//   online softmax in the log2 domain on the accumulator fragment (a lane holds 2 keys x 2 rows; the row maximum is
//               a butterfly over the 8 lanes that share the rows; the row sum is reduced once, at the end).
//   O^T = V^T P^T   m16n8k16, dims on the M side, keys on the contraction side.  A lane loads 16 bytes of four key
//               rows and pairs equal dims of two keys with byte permutes; P (bf16 hi + lo) moves from the accumulator
//               layout into the B layout with movmatrix.  The M position -> key assignment of the first product is
//               chosen so that this transposition lands every key where the permuted V fragment expects it.
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16_16816r(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// barrier among the two warps of a pair (ids 2 .. 5; 0 is the whole CTA, 1 the consumer warps)
__device__ __forceinline__ void pair_sync(int pair) { asm volatile("bar.sync %0, 64;" ::"r"(2 + pair) : "memory"); }

constexpr int ATT_TK = 16;                  // keys per tile
constexpr int ATT_DW = 64;                  // dims per warp
struct AttK { uint4 k[2][2]; };             // raw K bits of a tile: key rows mu(g), mu(g) + 2; 8 dims of each 32-dim block
struct AttV { uint4 v[4]; };                // raw V bits of a tile: key rows 4t .. 4t+3; dims 8g .. 8g+7 of the warp's 64
struct AttAcc {                             // running state of a unit's rows: lane (g, t) tracks rows 2t, 2t+1
    float o[4][4];                          // O^T tile e: [0],[1]: dim 8g + 2e, rows 2t, 2t+1; [2],[3]: dim 8g + 2e + 1
    float m[2], l[2];                       // running maximum (log2 domain) and this lane's share of the running sum
};
struct AttP { unsigned bh[2], bl[2]; float cf[2]; };    // a tile's probabilities in the B layout (bf16 hi, lo), rescale factors

template <int HD> struct AttSm {
    static constexpr int QS = HD * 2 + 64;                      // bytes per Q row (padded: two rows per shared-memory phase)
    static constexpr int Q_BYTES = 2 * M_MAX * QS;              // hi plane, lo plane
    static constexpr int MB_OFF = (Q_BYTES + 15) / 16 * 16;     // merge buffer [units][ATT_RB][ATT_MB_STRIDE] floats; while the
                                                                // tiles run, the pairs' score exchange [4][2][1 or 2][2][32] float4
};

// Page-table entries of a window of 32 pages, one per lane; a lane asks for the page of a key by shuffle.
struct PageWin {
    int first, pgs;
    __device__ __forceinline__ void load(const int* page_table, int n_pages, int first_page) {
        first = first_page;
        pgs = __ldg(page_table + min(first_page + (int)(threadIdx.x & 31), n_pages - 1));
    }
    // every lane calls this with its own key; the keys of one call lie within [first, first + 32) pages
    __device__ __forceinline__ int page_of(int key, int psh) const { return __shfl_sync(0xffffffffu, pgs, (key >> psh) - first); }
};

// kc / vc point at the warp's first dim of the head (element offset hh * HD + dim offset is added by the caller per row)
// A page number outside the cache never becomes an address: the access goes to page 0 and the state word records it.
__device__ __forceinline__ int checked_page(int pg, int n_pages, State* st, int where) {
    if ((unsigned)pg < (unsigned)n_pages) return pg;
    if (st) { atomicCAS(&st->status, 0, ST_INTERNAL); st->timeout_where = where; }
    return 0;
}

template <int HD>
__device__ __forceinline__ void att_load(AttK& tk, AttV& tv, const __nv_bfloat16* kc, const __nv_bfloat16* vc, const PageWin& pw,
                                         int H, int hh, int dof, int psh, int psm, int key0, int last_key, int n_pages, State* st) {
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int mu = 4 * (g >> 1) + (g & 1);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int key = min(key0 + mu + 2 * r, last_key);
        const int pg = checked_page(pw.page_of(key, psh), n_pages, st, 50);
        const __nv_bfloat16* row = kc + ((((size_t)pg * H + hh) << psh) + (key & psm)) * HD + dof + 8 * t;
        tk.k[r][0] = __ldcg(reinterpret_cast<const uint4*>(row));
        tk.k[r][1] = __ldcg(reinterpret_cast<const uint4*>(row + 32));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int key = min(key0 + 4 * t + i, last_key);
        const int pg = checked_page(pw.page_of(key, psh), n_pages, st, 51);
        const __nv_bfloat16* row = vc + ((((size_t)pg * H + hh) << psh) + (key & psm)) * HD + dof + 8 * g;
        tv.v[i] = __ldcg(reinterpret_cast<const uint4*>(row));
    }
}

// This warp's 64 dims of S = K Q^T for one tile: sc[0], sc[1]: key key0 + mu(g), rows 2t, 2t+1; sc[2], sc[3]: key + 2.
// qw: shared-memory address of the hi plane at this warp's first dim; row stride QS, lo plane M_MAX rows further.
template <int QS>
__device__ __forceinline__ void att_scores(const AttK& tk, float (&sc)[4], uint32_t qw, int row0) {
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const uint32_t qh = qw + (uint32_t)((row0 + g) * QS + 16 * t);
    const uint32_t ql = qh + (uint32_t)(M_MAX * QS);
    sc[0] = sc[1] = sc[2] = sc[3] = 0.f;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        uint4 h, l;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(h.x), "=r"(h.y), "=r"(h.z), "=r"(h.w) : "r"(qh + 64u * j));
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(l.x), "=r"(l.y), "=r"(l.z), "=r"(l.w) : "r"(ql + 64u * j));
        mma_bf16_16816r(sc, tk.k[0][j].x, tk.k[1][j].x, tk.k[0][j].y, tk.k[1][j].y, h.x, h.y);
        mma_bf16_16816r(sc, tk.k[0][j].x, tk.k[1][j].x, tk.k[0][j].y, tk.k[1][j].y, l.x, l.y);
        mma_bf16_16816r(sc, tk.k[0][j].z, tk.k[1][j].z, tk.k[0][j].w, tk.k[1][j].w, h.z, h.w);
        mma_bf16_16816r(sc, tk.k[0][j].z, tk.k[1][j].z, tk.k[0][j].w, tk.k[1][j].w, l.z, l.w);
    }
}

// Masking, online-softmax update and the probabilities of a tile in the layout the second product reads.
__device__ __forceinline__ void att_softmax(float (&sc)[4], AttAcc& ac, AttP& pp, int row0, int key0, int ke, int pos0) {
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int ka = key0 + 4 * (g >> 1) + (g & 1), kb2 = ka + 2;
    const int lim0 = pos0 + row0 + 2 * t, lim1 = lim0 + 1;            // last key rows 2t / 2t+1 may see
    if (ka >= ke || ka > lim0) sc[0] = -INFINITY;
    if (ka >= ke || ka > lim1) sc[1] = -INFINITY;
    if (kb2 >= ke || kb2 > lim0) sc[2] = -INFINITY;
    if (kb2 >= ke || kb2 > lim1) sc[3] = -INFINITY;
    float p[4];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float mx = fmaxf(sc[r], sc[2 + r]);
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        const float mn = fmaxf(ac.m[r], mx);
        pp.cf[r] = (ac.m[r] == -INFINITY) ? 0.f : ex2f(ac.m[r] - mn);
        p[r] = (sc[r] == -INFINITY) ? 0.f : ex2f(sc[r] - mn);
        p[2 + r] = (sc[2 + r] == -INFINITY) ? 0.f : ex2f(sc[2 + r] - mn);
        ac.l[r] = ac.l[r] * pp.cf[r] + (p[r] + p[2 + r]);
        ac.m[r] = mn;
    }
    // P as bf16 hi + lo, moved into the B layout: b0 = keys 4t, 4t+1 of row g; b1 = keys 4t+2, 4t+3
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        unsigned hi, lo;
        split_hi_lo(make_float2(p[2 * q], p[2 * q + 1]), hi, lo);
        pp.bh[q] = movmatrix_trans(hi);
        pp.bl[q] = movmatrix_trans(lo);
    }
}

// O^T += V^T P^T on this warp's 64 dims
__device__ __forceinline__ void att_accumulate(const AttV& tv, AttAcc& ac, const AttP& pp) {
    const unsigned w0[4] = {tv.v[0].x, tv.v[0].y, tv.v[0].z, tv.v[0].w};
    const unsigned w1[4] = {tv.v[1].x, tv.v[1].y, tv.v[1].z, tv.v[1].w};
    const unsigned w2[4] = {tv.v[2].x, tv.v[2].y, tv.v[2].z, tv.v[2].w};
    const unsigned w3[4] = {tv.v[3].x, tv.v[3].y, tv.v[3].z, tv.v[3].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        // dims 8g + 2e (M rows 0-7 of the instruction) and + 1 (M rows 8-15); keys (4t, 4t+1) then (4t+2, 4t+3)
        const unsigned a0 = __byte_perm(w0[e], w1[e], 0x5410), a1 = __byte_perm(w0[e], w1[e], 0x7632);
        const unsigned a2 = __byte_perm(w2[e], w3[e], 0x5410), a3 = __byte_perm(w2[e], w3[e], 0x7632);
        float (&o)[4] = ac.o[e];
        o[0] *= pp.cf[0]; o[1] *= pp.cf[1]; o[2] *= pp.cf[0]; o[3] *= pp.cf[1];
        mma_bf16_16816r(o, a0, a1, a2, a3, pp.bh[0], pp.bh[1]);
        mma_bf16_16816r(o, a0, a1, a2, a3, pp.bl[0], pp.bl[1]);
    }
}

// One work item of the tensor-core attention: head hh, split s of S (chunk_tiles tiles each) of the keys 0 .. pos0 + M - 1
// for the rows of `a`.  append: this pass's K / V rows are rotated, rounded and written to the cache by the item whose
// key range holds them (false: they are in the cache already).
template <int HD, bool DUAL = false>
__device__ __forceinline__ void att_item(const Dev& D, const AttArgs& a, Ctx& c, int hh, int s, int S, int chunk_tiles, bool append) {
    typedef __nv_bfloat16 WT;
    constexpr int NSPLIT = HD / ATT_DW;               // warps per unit: 1 (head_dim 64) or 2 (head_dim 128)
    constexpr int NUNITS = NWARPS / NSPLIT;
    constexpr int half = HD / 2;
    constexpr int QS = AttSm<HD>::QS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int H = D.dm.H, d = D.dm.d, psh = D.dm.ps_shift, psm = D.dm.page_size - 1;
    const int M = a.M, pos0 = a.pos0;
    const int T = pos0 + M;
    const int ntiles_all = (T + ATT_TK - 1) / ATT_TK;
    const int R = (M + 7) >> 3;                       // row groups of 8
    // DUAL (prompt pass, two row groups): every unit works on both row groups of its tiles, two independent chains of
    // dependent instructions side by side; else a unit owns one row group
    constexpr int NRG = DUAL ? 2 : 1;
    const int nw = DUAL ? NUNITS : NUNITS / R;        // units that share the tiles of an item (a power of two)
    const int tpw = (chunk_tiles + nw - 1) / nw;
    const float qscale = rsqrtf((float)HD) * 1.4426950408889634f;      // 1/sqrt(hd) and log2(e)
    WT* kc = reinterpret_cast<WT*>(a.kc);
    WT* vc = reinterpret_cast<WT*>(a.vc);
    unsigned char* qs = reinterpret_cast<unsigned char*>(c.smem + WORK_OFF);
    float* mb = reinterpret_cast<float*>(c.smem + WORK_OFF + AttSm<HD>::MB_OFF);
    const int unit = warp / NSPLIT, hsel = warp % NSPLIT, dof = hsel * ATT_DW;
    const int rg = DUAL ? 0 : unit % R, tlane = DUAL ? unit : unit / R;
    const int row0 = rg * 8;
    const uint32_t qw = smem_u32(qs) + (uint32_t)(dof * 2);
    // rows >= M of the row groups in use are zero in both planes
    for (int idx = tid; idx < (8 * R - M) * half; idx += NTHREADS) {
        const int i = M + idx / half, e = idx % half;
        reinterpret_cast<unsigned*>(qs + (size_t)i * QS)[e] = 0u;
        reinterpret_cast<unsigned*>(qs + (size_t)(M_MAX + i) * QS)[e] = 0u;
    }
    const int tb = s * chunk_tiles, te = min(ntiles_all, tb + chunk_tiles);
    const int kb = tb * ATT_TK, ke = min(T, te * ATT_TK);
    // this pass's rows: q rotated, scaled and split into the bf16 hi / lo planes; k rotated and, with v, rounded and
    // appended to the cache when the row's position lies in my key range.  One cos / sin pair serves q and k, and
    // all six loads of an element are issued before the first is used.
    for (int idx = tid; idx < M * half; idx += NTHREADS) {
        const int i = idx / half, e = idx % half, pos = pos0 + i;
        const float* src = a.qkv + (size_t)i * 3 * d + hh * HD + e;
        const float q1 = ldcg_f(src), q2 = ldcg_f(src + half);
        const float k1 = ldcg_f(src + d), k2 = ldcg_f(src + d + half);
        const float v1 = ldcg_f(src + 2 * d), v2 = ldcg_f(src + 2 * d + half);
        const int page = checked_page(__ldg(D.page_table + (pos >> psh)), D.dm.n_phys, D.st, 52);
        float cs, sn; rope_cs(D, pos, e, cs, sn);
        const float r1 = (q1 * cs - q2 * sn) * qscale, r2 = (q2 * cs + q1 * sn) * qscale;
        const __nv_bfloat16 h1 = __float2bfloat16_rn(r1), h2 = __float2bfloat16_rn(r2);
        __nv_bfloat16* ph = reinterpret_cast<__nv_bfloat16*>(qs + (size_t)i * QS);
        __nv_bfloat16* pl = reinterpret_cast<__nv_bfloat16*>(qs + (size_t)(M_MAX + i) * QS);
        ph[e] = h1; ph[e + half] = h2;
        pl[e] = __float2bfloat16_rn(r1 - __bfloat162float(h1)); pl[e + half] = __float2bfloat16_rn(r2 - __bfloat162float(h2));
        if (append && pos >= kb && pos < ke) {
            const size_t base = ((((size_t)page * H + hh) << psh) + (pos & psm)) * HD;
            kc[base + e] = __float2bfloat16_rn(k1 * cs - k2 * sn);
            kc[base + e + half] = __float2bfloat16_rn(k2 * cs + k1 * sn);
            vc[base + e] = __float2bfloat16_rn(v1);
            vc[base + e + half] = __float2bfloat16_rn(v2);
        }
    }
    AttAcc ac[NRG];
#pragma unroll
    for (int r = 0; r < NRG; ++r) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { ac[r].o[e][0] = ac[r].o[e][1] = ac[r].o[e][2] = ac[r].o[e][3] = 0.f; }
        ac[r].m[0] = ac[r].m[1] = -INFINITY; ac[r].l[0] = ac[r].l[1] = 0.f;
    }
    // this unit's tiles: a contiguous run, so that one window of page-table entries serves many of them
    int tile = tb + tlane * tpw;
    const int tend = min(te, tile + tpw);
    PageWin pw;
    if (tile < tend) pw.load(D.page_table, D.dm.n_pages, (tile * ATT_TK) >> psh);
    cta_sync();
    auto fetch = [&](AttK& tk, AttV& tv, int ti) {
        const int key0 = ti * ATT_TK, key1 = min(key0 + ATT_TK - 1, T - 1);
        if ((key1 >> psh) - pw.first >= 32) pw.load(D.page_table, D.dm.n_pages, key0 >> psh);
        att_load<HD>(tk, tv, kc, vc, pw, H, hh, dof, psh, psm, key0, T - 1, D.dm.n_phys, D.st);
    };
    AttP pp[NRG];
    auto step = [&](const AttK& tk, const AttV& tv, int ti) {
        float sc[NRG][4];
#pragma unroll
        for (int r = 0; r < NRG; ++r) att_scores<QS>(tk, sc[r], qw, row0 + 8 * r);
        if constexpr (NSPLIT == 2) {
            // the pair's halves of the dot products meet in shared memory (two buffers, used alternately)
            float4* xb = reinterpret_cast<float4*>(mb) + (size_t)((unit * 2 + (ti & 1)) * NRG * 2) * 32;
#pragma unroll
            for (int r = 0; r < NRG; ++r) xb[(r * 2 + hsel) * 32 + lane] = make_float4(sc[r][0], sc[r][1], sc[r][2], sc[r][3]);
            pair_sync(unit);
#pragma unroll
            for (int r = 0; r < NRG; ++r) {
                const float4 ot = xb[(r * 2 + (hsel ^ 1)) * 32 + lane];
                sc[r][0] += ot.x; sc[r][1] += ot.y; sc[r][2] += ot.z; sc[r][3] += ot.w;
            }
        }
#pragma unroll
        for (int r = 0; r < NRG; ++r) att_softmax(sc[r], ac[r], pp[r], row0 + 8 * r, ti * ATT_TK, ke, pos0);
#pragma unroll
        for (int r = 0; r < NRG; ++r) att_accumulate(tv, ac[r], pp[r]);
    };
    // One register set for K and V (a second one would not fit: the register allocation is shared with the
    // linear operators).  A tile therefore costs a memory latency; the split count above keeps the run of
    // tiles per unit short, and the other units and CTAs keep the memory system busy meanwhile.  (In the prompt
    // pass, where a unit walks over hundreds of tiles, requesting the next tile early was measured: 2 % slower.)
    AttK k0;
    AttV v0;
    while (tile < tend) {
        fetch(k0, v0, tile);
        step(k0, v0, tile);
        ++tile;
    }
    // the row sums: lanes that share rows add their shares in a fixed order
#pragma unroll
    for (int q = 0; q < NRG; ++q) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            ac[q].l[r] += __shfl_xor_sync(0xffffffffu, ac[q].l[r], 4);
            ac[q].l[r] += __shfl_xor_sync(0xffffffffu, ac[q].l[r], 8);
            ac[q].l[r] += __shfl_xor_sync(0xffffffffu, ac[q].l[r], 16);
        }
    }
    if constexpr (NSPLIT == 2) cta_sync();          // the merge buffer lies over the pairs' exchange buffers
    // merge the units of a row group through shared memory, four rows at a time
#pragma unroll
    for (int rb = 0; rb < M_MAX / ATT_RB; ++rb) {
        if (rb * ATT_RB >= M) break;
        const int nr = min(ATT_RB, M - rb * ATT_RB);
        const AttAcc& aa = ac[NRG == 2 ? (rb >> 1) : 0];
        if ((DUAL || rg == (rb >> 1)) && (t >> 1) == (rb & 1)) {
            const int rl = 2 * (t & 1);
            float* r0 = mb + ((size_t)tlane * ATT_RB + rl) * ATT_MB_STRIDE;
            float* r1 = r0 + ATT_MB_STRIDE;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int dd = dof + 8 * g + 2 * e;
                *reinterpret_cast<float2*>(r0 + dd) = make_float2(aa.o[e][0], aa.o[e][2]);
                *reinterpret_cast<float2*>(r1 + dd) = make_float2(aa.o[e][1], aa.o[e][3]);
            }
            if (g == 0 && hsel == 0) { r0[HD_MAX] = aa.m[0]; r0[HD_MAX + 1] = aa.l[0]; r1[HD_MAX] = aa.m[1]; r1[HD_MAX + 1] = aa.l[1]; }
        }
        cta_sync();
        for (int idx = tid; idx < nr * HD; idx += NTHREADS) {
            const int r = idx / HD, e = idx % HD, i = rb * ATT_RB + r;
            float mx = -INFINITY;
            for (int w = 0; w < nw; ++w) mx = fmaxf(mx, mb[((size_t)w * ATT_RB + r) * ATT_MB_STRIDE + HD_MAX]);
            float den = 0.f, num = 0.f;
            for (int w = 0; w < nw; ++w) {
                const float* row = mb + ((size_t)w * ATT_RB + r) * ATT_MB_STRIDE;
                const float mw = row[HD_MAX];
                if (mw != -INFINITY) {
                    const float wgt = ex2f(mw - mx);
                    den += row[HD_MAX + 1] * wgt;
                    num += row[e] * wgt;
                }
            }
            if (S == 1) {
                const float ov = num / den;
                a.out[(size_t)i * d + hh * HD + e] = ov;
                if (a.opk) pk_store(a.opk + (size_t)i * d * 4, hh * HD + e, ov);
            } else {
                D.att_po[(((size_t)i * H + hh) * S_CAP + s) * HD + e] = num;
                if (e == 0) {
                    D.att_ml[(((size_t)i * H + hh) * S_CAP + s) * 2 + 0] = mx;
                    D.att_ml[(((size_t)i * H + hh) * S_CAP + s) * 2 + 1] = den;
                }
            }
        }
        cta_sync();
    }
    if (S > 1) {
        // the partials of this CTA are ordered before the counter by the barrier above and the release of the
        // atomic; the last arriver's acquire orders the counter before its reads of every split's partials
        if (tid == 0) {
            unsigned prev;
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(D.att_cnt + hh) : "memory");
            const int last = (prev == (unsigned)(S - 1));
            c.ctl->att_last = last;
            if (last) D.att_cnt[hh] = 0u;
        }
        cta_sync();
        if (*(volatile int*)&c.ctl->att_last) {
            if (S <= 4) att_merge_splits<4, 4>(D, a, hh, S, M);
            else if (S <= 8) att_merge_splits<8, 2>(D, a, hh, S, M);
            else att_merge_splits<S_CAP, 1>(D, a, hh, S, M);
        }
        cta_sync();
    }
}

template <int HD>
__device__ __noinline__ void attention_mma(const Dev& D, const AttArgs& a, Ctx& c) {
    constexpr int NUNITS = NWARPS / (HD / ATT_DW);
    const int H = D.dm.H;
    const int ntiles_all = (a.pos0 + a.M + ATT_TK - 1) / ATT_TK;
    const int nw = NUNITS / ((a.M + 7) >> 3);
    const int nw_sh = 31 - __clz(nw);
    // KV splits per head.  An item costs its units' tiles (one memory latency each) plus a fixed part, and a head
    // that is split pays for the merge of its partials through global memory (several dependent round trips, about
    // as long as three tiles): very short caches stay unsplit.
    int S = 1;
    {
        const float inv_ctas = 1.0f / (float)c.nctas;
        float best = -1.f;
#pragma unroll
        for (int sc = 1; sc <= S_CAP; ++sc) {
            const int chunk_ = (ntiles_all + sc - 1) / sc;
            const int tpw_ = (chunk_ + nw - 1) >> nw_sh;
            const float waves = ceilf((float)(H * sc) * inv_ctas - 1e-4f);
            const float cost = waves * (float)(tpw_ + 2 + (sc > 1 ? 3 : 0));
            if ((sc == 1 || chunk_ >= 2) && (best < 0.f || cost < best)) { best = cost; S = sc; }
        }
    }
    const int chunk_tiles = (ntiles_all + S - 1) / S;
    for (int item = c.cta; item < H * S; item += c.nctas) att_item<HD>(D, a, c, item / S, item % S, S, chunk_tiles, true);
}

// The prompt pass: `nrows` rows at positions a.pos0.. whose K / V are in the cache already; an item is a block of 16
// rows of one head against all keys it may see (no splits: there are plenty of items).
template <int HD>
__device__ __noinline__ void attention_prefill(const Dev& D, const AttArgs& a, Ctx& c, int nrows) {
    const int H = D.dm.H, d = D.dm.d;
    const int nblk = (nrows + M_MAX - 1) / M_MAX;
    for (int item = c.cta; item < nblk * H; item += c.nctas) {
        const int rb = item / H, hh = item % H;
        AttArgs b = a;
        b.qkv = a.qkv + (size_t)rb * M_MAX * 3 * d;
        b.out = a.out + (size_t)rb * M_MAX * d;
        b.opk = nullptr;
        b.M = min(M_MAX, nrows - rb * M_MAX);
        b.pos0 = a.pos0 + rb * M_MAX;
        // full blocks of 16 rows: both row groups in every unit; a shorter last block: the decode path's split
        if (b.M > 8) att_item<HD, true>(D, b, c, hh, 0, 1, (b.pos0 + b.M + ATT_TK - 1) / ATT_TK, false);
        else att_item<HD, false>(D, b, c, hh, 0, 1, (b.pos0 + b.M + ATT_TK - 1) / ATT_TK, false);
    }
}
static_assert(AttSm<HD_MAX>::MB_OFF + NWARPS * ATT_RB * ATT_MB_STRIDE * 4 <= WORK_BYTES, "tensor-core attention buffers do not fit in the work area");
static_assert(4 * 2 * 2 * 2 * 32 * 16 <= NWARPS * ATT_RB * ATT_MB_STRIDE * 4, "the score exchange of two row groups does not fit in the merge buffer");

template <typename WT>
__device__ __forceinline__ void attention_op(const Dev& D, const AttArgs* sa, Ctx& c) {
    // sa points into the consumers' operator table in shared memory
    if constexpr (sizeof(WT) == 2) {
        if (D.dm.hd == 128) { attention_mma<128>(D, *sa, c); return; }
        if (D.dm.hd == 64) { attention_mma<64>(D, *sa, c); return; }
    }
    if (D.dm.hd == 128) attention_impl<WT, 4>(D, *sa, c);
    else if (D.dm.hd == 64) attention_impl<WT, 2>(D, *sa, c);
    else attention_impl<WT, 1>(D, *sa, c);
}

static_assert((M_MAX * HD_MAX + NWARPS * ATT_RB * ATT_MB_STRIDE + NWARPS * 40) * 4 <= WORK_BYTES, "attention buffers do not fit in the work area");

}  // namespace kg
