// Host side of the C ABI declared in include/kangaroo.h: arena layout, synthetic weight fill,
// launches of the persistent decode kernel, small result copies.  No device allocation anywhere.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/kangaroo.h"
#include "kg_engine.cuh"
#include "kg_prefill.cuh"

using namespace kg;

// ------------------------------------------------------------------------------------ generator
// Counter-based generator, implemented here independently of the host-side test generator:
//   base = mix(mix(seed) + tid); u = mix(base + i); g = bytesum(u) - 1020; x = float(g) * scale.
// mix is the SplitMix64 output function (Steele, Lea, Flood).
namespace {

__host__ __device__ inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
inline uint64_t stream_base(uint64_t seed, uint64_t tid) { return mix64(mix64(seed) + tid); }
inline float gen_scale(double std_) { return (float)(std_ / std::sqrt(43690.0)); }

__device__ __forceinline__ float gen_value(uint64_t base, uint64_t i, float scale) {
    const uint64_t u = mix64(base + i);
    const unsigned lo = (unsigned)u, hi = (unsigned)(u >> 32);
    // byte sum via two SIMD-in-register adds
    const unsigned s2 = (lo & 0x00ff00ffu) + ((lo >> 8) & 0x00ff00ffu) + (hi & 0x00ff00ffu) + ((hi >> 8) & 0x00ff00ffu);
    const int g = (int)((s2 & 0xffffu) + (s2 >> 16)) - 1020;
    return __fmul_rn((float)g, scale);
}

template <typename WT>
__global__ void fill_matrix_kernel(WT* out, uint64_t base, uint64_t count, float scale) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = float_to_wt<WT>(gen_value(base, i, scale));
}
__global__ void fill_gain_kernel(float* out, uint64_t base, int count, float scale) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x)
        out[i] = __fadd_rn(1.0f, gen_value(base, (uint64_t)i, scale));
}
__global__ void fill_f32_kernel(float* out, uint64_t base, uint64_t count, float scale) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = gen_value(base, i, scale);
}
// KV cache entries for positions [0, T): element index (pos*H + head)*hd + e of the stream.
template <typename WT>
__global__ void fill_cache_kernel(WT* cache, const int* page_table, uint64_t base, int T, int H, int hd, int ps, float scale) {
    const uint64_t count = (uint64_t)T * H * hd;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (uint64_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % hd), head = (int)((i / hd) % H), pos = (int)(i / ((uint64_t)hd * H));
        const size_t dst = (((size_t)page_table[pos / ps] * H + head) * ps + pos % ps) * hd + e;
        cache[dst] = float_to_wt<WT>(gen_value(base, i, scale));
    }
}
__global__ void fill_tokens_kernel(int* out, uint64_t base, int count, int vocab) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x)
        out[i] = (int)(mix64(base + (uint64_t)i) % (uint64_t)vocab);
}

// fp32 rows -> packed rows (scaled by gain) + per-slice sums of squares, sliced over the columns exactly as the
// CTAs of the decode kernel slice an operator's output (slice c = columns [K c / n, K (c+1) / n)).
__global__ void pack_rows_kernel(const float* x, int ldx, int M, int K, const float* gain, unsigned char* xpk, int ldpk,
                                 float* ssq, int nslices) {
    __shared__ float sred[8];
    const int cta = blockIdx.x;
    const int k0 = (int)((unsigned)K * (unsigned)cta / (unsigned)nslices), k1 = (int)((unsigned)K * (unsigned)(cta + 1) / (unsigned)nslices);
    for (int m = 0; m < M; ++m) {
        float ss = 0.f;
        for (int k = k0 + threadIdx.x; k < k1; k += blockDim.x) {
            const float v = x[(size_t)m * ldx + k];
            ss += v * v;
            pk_store(xpk + (size_t)m * ldpk, k, gain ? v * gain[k] : v);
        }
        ss = warp_sum(ss);
        if ((threadIdx.x & 31) == 0) sred[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0 && ssq) {
            float t = 0.f;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sred[w];
            ssq[(size_t)m * nslices + cta] = t;
        }
        __syncthreads();
    }
}

enum { TID_EMBED = 1, TID_HEAD = 2, TID_PROMPT = 3, TID_HIDDEN = 4, TID_GFINAL = 6, TID_DRAFT = 7, TID_LAYER_BASE = 100 };
enum { K_WQKV = 0, K_WO = 1, K_WGATE = 2, K_WUP = 3, K_WDOWN = 4, K_G1 = 5, K_G2 = 6, K_KCACHE = 8, K_VCACHE = 9 };
inline uint64_t layer_tid(int layer, int k) { return (uint64_t)TID_LAYER_BASE + 16ull * (uint64_t)layer + (uint64_t)k; }

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t off_hApk, off_hBpk, off_attnpk, off_actpk, off_featApk, off_featDpk, off_abufpk, off_ssqA, off_ssqB, off_ssqF, off_ssqAb;
    size_t off_layers, off_pt, off_kc, off_vc, off_h, off_feat, off_abuf, off_qkv, off_attn, off_act, off_po, off_ml,
        off_cnt, off_hp, off_dbgd, off_dbgv, off_out, off_S, off_rlog, off_prompt, off_st, off_bar;
    // tensor-core prompt pass (0 bytes each when the shape cannot take it)
    size_t off_pf_h, off_pf_h2, off_pf_qkv, off_pf_attn, off_pf_gate, off_pf_up, off_pf_hi, off_pf_lo, off_pf_err;
    size_t off_embed, off_head, off_gfinal;
    std::vector<size_t> off_w[5];     // wqkv, wo, wgate, wup, wdown
    std::vector<size_t> off_g[2];
    size_t total;
};

// The tensor-core prompt pass needs bf16 weights, a head_dim the tensor-core attention knows, and matrix sides that
// are whole tiles: N a multiple of 128, K a multiple of 64.
bool prefill_tc_shape(const kg_config* c) {
    return c->dtype == KG_BF16 && (c->head_dim == 64 || c->head_dim == 128) && c->d_model % 128 == 0 && c->d_ffn % 128 == 0 &&
           c->d_model <= PF_EW_THREADS * 4 * PF_NORM_V;      // the norm kernel keeps a row in registers
}

bool valid_config(const kg_config* c) {
    if (!c || c->struct_size != sizeof(kg_config)) return false;
    if (c->n_layers < 2 || c->exit_layer < 1 || c->exit_layer >= c->n_layers) return false;
    if (c->d_model <= 0 || c->n_heads <= 0 || c->n_heads * c->head_dim != c->d_model) return false;
    if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->d_model % 8 || c->d_ffn % 8 || c->d_ffn <= 0 || c->vocab <= 1) return false;
    if (c->dtype != KG_F32 && c->dtype != KG_BF16) return false;
    if (c->gamma_max < 1 || c->gamma_max > KG_GAMMA_MAX) return false;
    if (c->page_size < 1 || (c->page_size & (c->page_size - 1)) || c->max_seq < 2) return false;       // pages hold a power of two of tokens
    if (c->n_heads > 256) return false;
    if (c->vocab > (1 << 20) || c->d_ffn > (1 << 20)) return false;      // rows x CTAs must fit 32 bits
    // one launch may run max_seq tokens, each at most 5 (L + 1) + 8 grid barriers of at most 1024 CTAs: the arrival
    // counter (31 bits beside the abort flag) must hold them all
    if ((long long)c->max_seq * (5LL * (c->n_layers + 1) + 8) * 1024LL >= (1LL << 31)) return false;
    // the plain path stages all rows of an operand in shared memory
    const int kmax = c->d_ffn > c->d_model ? c->d_ffn : c->d_model;
    const bool plain_somewhere = c->dtype == KG_F32 || (c->d_model % 16) || (c->d_ffn % 16);
    if (plain_somewhere && (size_t)kmax * KG_M_MAX * 4 > (size_t)SIMPLE_XS_BYTES) return false;
    return true;
}

Layout make_layout(const kg_config* c, int own_weights, int nctas) {
    Layout L;
    const size_t es = c->dtype == KG_BF16 ? 2 : 4;
    const size_t d = c->d_model, F = c->d_ffn, V = c->vocab, H = c->n_heads, hd = c->head_dim;
    const int nl = c->n_layers;
    const size_t n_pages = (c->max_seq + c->page_size - 1) / c->page_size;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
    L.off_st = take(sizeof(State));
    L.off_bar = take(256);
    L.off_layers = take(sizeof(LayerW) * (nl + 1));
    L.off_pt = take(sizeof(int) * n_pages);
    const size_t cache_bytes = (size_t)(nl + 1) * n_pages * H * c->page_size * hd * es;
    L.off_kc = take(cache_bytes);
    L.off_vc = take(cache_bytes);
    L.off_h = take(4 * KG_M_MAX * d);
    L.off_feat = take(4 * (KG_M_MAX + 1) * d);
    L.off_abuf = take(4 * 2 * d);
    L.off_qkv = take(4 * KG_M_MAX * 3 * d);
    L.off_attn = take(4 * KG_M_MAX * d);
    L.off_act = take(4 * KG_M_MAX * F);
    L.off_hApk = take(4 * KG_M_MAX * d);
    L.off_hBpk = take(4 * KG_M_MAX * d);
    L.off_attnpk = take(4 * KG_M_MAX * d);
    L.off_actpk = take(4 * KG_M_MAX * F);
    L.off_featApk = take(4 * (KG_M_MAX + 1) * d);
    L.off_featDpk = take(4 * (KG_M_MAX + 1) * d);
    L.off_abufpk = take(4 * 2 * d);
    L.off_ssqA = take(4 * (size_t)KG_M_MAX * nctas);
    L.off_ssqB = take(4 * (size_t)KG_M_MAX * nctas);
    L.off_ssqF = take(4 * (size_t)(KG_M_MAX + 1) * nctas);
    L.off_ssqAb = take(4 * (size_t)2 * nctas);
    L.off_po = take(4 * (size_t)KG_M_MAX * H * S_CAP * hd);
    L.off_ml = take(4 * (size_t)KG_M_MAX * H * S_CAP * 2);
    L.off_cnt = take(4 * H);
    L.off_hp = take(sizeof(float4) * (size_t)nctas * KG_M_MAX);
    L.off_dbgd = take(c->debug_logits ? 4 * (size_t)KG_M_MAX * V : 0);
    L.off_dbgv = take(c->debug_logits ? 4 * (size_t)KG_M_MAX * V : 0);
    L.off_out = take(4 * (size_t)(c->max_seq + KG_M_MAX));
    L.off_S = take(4 * (size_t)(c->max_seq + KG_M_MAX));
    L.off_rlog = take(16 * (size_t)(c->max_seq + KG_M_MAX));
    L.off_prompt = take(4 * (size_t)c->max_seq);
    {
        const size_t R = prefill_tc_shape(c) ? (size_t)PF_ROWS : 0, kmax = F > d ? F : d;
        L.off_pf_h = take(4 * R * d); L.off_pf_h2 = take(4 * R * d); L.off_pf_qkv = take(4 * R * 3 * d);
        L.off_pf_attn = take(4 * R * d); L.off_pf_gate = take(4 * R * F); L.off_pf_up = take(4 * R * F);
        L.off_pf_hi = take(2 * R * kmax); L.off_pf_lo = take(2 * R * kmax); L.off_pf_err = take(R ? 64 + 4 * R : 0);      // error word, then 1/rms per row
    }
    for (int k = 0; k < 5; ++k) L.off_w[k].assign(nl + 1, 0);
    for (int k = 0; k < 2; ++k) L.off_g[k].assign(nl + 1, 0);
    L.off_embed = L.off_head = L.off_gfinal = 0;
    if (own_weights) {
        L.off_embed = take(es * V * d);
        L.off_head = take(es * V * d);
        L.off_gfinal = take(4 * d);
        for (int i = 0; i <= nl; ++i) {
            L.off_w[K_WQKV][i] = take(es * 3 * d * d);
            L.off_w[K_WO][i] = take(es * d * d);
            if (i < nl) {
                L.off_w[K_WGATE][i] = take(es * F * d);
                L.off_w[K_WUP][i] = take(es * F * d);
                L.off_w[K_WDOWN][i] = take(es * d * F);
            }
            L.off_g[0][i] = take(4 * d);
            L.off_g[1][i] = take(4 * d);
        }
    }
    L.total = o;
    return L;
}

// SM count of the current device (one CTA per SM in every launch), looked up once per device.
constexpr int MAX_DEVICES = 64;
int g_sm_count[MAX_DEVICES] = {0};
int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev >= 0 && dev < MAX_DEVICES && g_sm_count[dev] > 0) return g_sm_count[dev];
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    if (dev >= 0 && dev < MAX_DEVICES) g_sm_count[dev] = n;
    return n;
}

// Device pointers handed in by the caller feed 16-byte bulk copies and vector loads: anything less aligned would
// fault on the device, so it is refused on the host.
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Token ids that arrive in device memory cannot be checked on the host: one thread per id records an argument
// error in the state word (the embedding lookup itself keeps every access in bounds).
__global__ void check_tokens_kernel(const int* toks, int n, int vocab, State* st) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && (unsigned)toks[i] >= (unsigned)vocab) atomicCAS(&st->status, 0, (int)KG_E_ARG);
}

}  // namespace

struct kg_model {
    kg_config cfg;
    Dev dev;
    Layout lay;
    char* arena;
    cudaStream_t stream;
    int nctas;
    size_t smem;
    bool own_weights;
    bool prefilled, pending, ar_used, dead;
    int prefill_mode;              // 0: tensor-core prompt pass when the shape and the prompt allow, 1: always the chunked pass
    unsigned long long wait_clk;   // budget of a device-side wait, in SM clocks
    int skip_arrival;              // test hook, consumed by the next launch
    cudaEvent_t ev0, ev1;          // timing of the decode loop in kg_generate, created on first use
    int gamma_pending;
    long long P_upper;      // upper bound of the device-side position P
    int force_simple;
    std::vector<LayerW> layers_host;
};

// Name and text of the CUDA error behind the last KG_E_CUDA of this thread ("" if there was none).
static thread_local char g_cuda_err[160] = "";
static bool cuda_failed(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return false;
    std::snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
    return true;
}
#define CK(x) do { if (cuda_failed((x), #x)) return KG_E_CUDA; } while (0)

extern "C" const char* kg_last_cuda_error(void) { return g_cuda_err; }

extern "C" const char* kg_strerror(int s) {
    switch (s) {
        case KG_OK: return "ok";
        case KG_E_ARG: return "invalid argument";
        case KG_E_STATE: return "call order violated";
        case KG_E_NOMEM: return "arena too small";
        case KG_E_SEQ_FULL: return "sequence would exceed max_seq";
        case KG_E_CUDA: return "CUDA runtime error";
        case KG_E_TIMEOUT: return "device-side wait timed out";
        case KG_E_LIMIT: return "size beyond the capacity of the library's static scratch (or of the operator scratch)";
        case KG_E_INTERNAL: return "a device-side index check failed (the access was skipped)";
        default: return "unknown status";
    }
}

extern "C" size_t kg_workspace_bytes(const kg_config* cfg, int own_weights) {
    if (!valid_config(cfg)) return 0;
    return make_layout(cfg, own_weights, sm_count()).total + 256;
}

template <typename WT>
static int launch_program(kg_model* m, const Program& pg) {
    CK(cudaMemsetAsync(m->dev.bar, 0, BAR_BYTES, m->stream));
    Program p = pg;
    p.force_simple = m->force_simple;
    p.wait_clk = m->wait_clk;
    p.skip_arrival = m->skip_arrival;
    m->skip_arrival = 0;
    void* args[] = {(void*)&m->dev, (void*)&p};
    CK(cudaLaunchCooperativeKernel((const void*)kg_persistent_kernel<WT>, dim3(m->nctas), dim3(DECODE_THREADS), args, m->smem, m->stream));
    return KG_OK;
}
static int launch(kg_model* m, const Program& pg) {
    return m->cfg.dtype == KG_BF16 ? launch_program<__nv_bfloat16>(m, pg) : launch_program<float>(m, pg);
}

static int read_state(kg_model* m, State* out) {
    CK(cudaMemcpyAsync(out, m->dev.st, sizeof(State), cudaMemcpyDeviceToHost, m->stream));
    CK(cudaStreamSynchronize(m->stream));
    if (out->status == ST_TIMEOUT) { m->dead = true; return KG_E_TIMEOUT; }
    if (out->status == ST_INTERNAL) {
        std::snprintf(g_cuda_err, sizeof(g_cuda_err), "device-side index check %d failed", out->timeout_where);
        m->dead = true;
        return KG_E_INTERNAL;
    }
    if (out->status != 0) {
        // an argument error found on the device (a token id outside the vocabulary): the sequence is unusable until
        // kg_reset, which also clears the state word; the weights are untouched
        m->prefilled = m->pending = false; m->ar_used = true;
        return out->status;
    }
    return KG_OK;
}

template <typename WT>
static int fill_weights(kg_model* m) {
    const kg_config& c = m->cfg;
    cudaStream_t s = m->stream;
    const uint64_t d = c.d_model, F = c.d_ffn, V = c.vocab;
    const int nl = c.n_layers;
    auto fill = [&](size_t off, uint64_t tid, uint64_t count, double std_) {
        fill_matrix_kernel<WT><<<1184, 256, 0, s>>>(reinterpret_cast<WT*>(m->arena + off), stream_base(c.seed, tid), count, gen_scale(std_));
    };
    auto gain = [&](size_t off, uint64_t tid) {
        fill_gain_kernel<<<16, 256, 0, s>>>(reinterpret_cast<float*>(m->arena + off), stream_base(c.seed, tid), (int)d, gen_scale(c.gain_std));
    };
    fill(m->lay.off_embed, TID_EMBED, V * d, c.embed_std);
    fill(m->lay.off_head, TID_HEAD, V * d, c.init_std);
    gain(m->lay.off_gfinal, TID_GFINAL);
    for (int i = 0; i <= nl; ++i) {
        const bool adapter = i == nl;
        const double os = adapter ? c.adapter_resid_scale : (i >= c.exit_layer ? c.deep_resid_scale : 1.0);
        // the output-projection std is formed in fp32 exactly as the host recipe does: float(init_std) * float(scale)
        const double std_o = (double)c.init_std * os;
        fill(m->lay.off_w[K_WQKV][i], layer_tid(i, K_WQKV), 3 * d * d, c.init_std);
        fill(m->lay.off_w[K_WO][i], layer_tid(i, K_WO), d * d, std_o);
        if (!adapter) {
            fill(m->lay.off_w[K_WGATE][i], layer_tid(i, K_WGATE), F * d, c.init_std);
            fill(m->lay.off_w[K_WUP][i], layer_tid(i, K_WUP), F * d, c.init_std);
            fill(m->lay.off_w[K_WDOWN][i], layer_tid(i, K_WDOWN), d * F, std_o);
        }
        gain(m->lay.off_g[0][i], layer_tid(i, K_G1));
        gain(m->lay.off_g[1][i], layer_tid(i, K_G2));
    }
    CK(cudaGetLastError());
    return KG_OK;
}

extern "C" int kg_init_model(const kg_config* cfg, const kg_weights* w, void* arena_dev, size_t arena_bytes,
                             void* cuda_stream, kg_model** out) {
    if (!out) return KG_E_ARG;
    *out = nullptr;
    if (!valid_config(cfg) || !arena_dev) return KG_E_ARG;
    if (w) {
        if (!w->embed_dev || !w->head_dev || !w->g_final_dev || !w->wqkv_dev || !w->wo_dev || !w->wgate_dev ||
            !w->wup_dev || !w->wdown_dev || !w->g1_dev || !w->g2_dev) return KG_E_ARG;
        if (!aligned16(w->embed_dev) || !aligned16(w->head_dev) || !aligned16(w->g_final_dev)) return KG_E_ARG;
        for (int i = 0; i <= cfg->n_layers; ++i) {
            const bool layer = i < cfg->n_layers;
            if (!w->wqkv_dev[i] || !w->wo_dev[i] || !w->g1_dev[i] || !w->g2_dev[i] ||
                (layer && (!w->wgate_dev[i] || !w->wup_dev[i] || !w->wdown_dev[i]))) return KG_E_ARG;
            if (!aligned16(w->wqkv_dev[i]) || !aligned16(w->wo_dev[i]) || !aligned16(w->g1_dev[i]) || !aligned16(w->g2_dev[i]) ||
                (layer && (!aligned16(w->wgate_dev[i]) || !aligned16(w->wup_dev[i]) || !aligned16(w->wdown_dev[i])))) return KG_E_ARG;
        }
    }
    const int nctas = sm_count();
    const int own = w ? 0 : 1;
    Layout lay = make_layout(cfg, own, nctas);
    char* base = reinterpret_cast<char*>(align_up(reinterpret_cast<size_t>(arena_dev), 256));
    if ((size_t)(base - reinterpret_cast<char*>(arena_dev)) + lay.total > arena_bytes) return KG_E_NOMEM;

    kg_model* m = new (std::nothrow) kg_model();
    if (!m) return KG_E_NOMEM;
    m->cfg = *cfg; m->lay = lay; m->arena = base; m->stream = (cudaStream_t)cuda_stream; m->nctas = nctas;
    m->own_weights = own != 0; m->prefilled = m->pending = m->ar_used = m->dead = false;
    m->gamma_pending = 0; m->P_upper = 0; m->force_simple = 0;
    m->wait_clk = WAIT_TIMEOUT_CLK; m->skip_arrival = 0; m->ev0 = m->ev1 = nullptr; m->prefill_mode = 0;
    m->smem = SMEM_TOTAL;

    const bool bf = cfg->dtype == KG_BF16;
    const void* kfn = bf ? (const void*)kg_persistent_kernel<__nv_bfloat16> : (const void*)kg_persistent_kernel<float>;
    if (cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m->smem) != cudaSuccess) { delete m; return KG_E_CUDA; }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kfn, DECODE_THREADS, m->smem) != cudaSuccess || occ < 1) { delete m; return KG_E_CUDA; }
    {
        // the kernel's warpgroups re-divide the registers the launch gives the CTA; a budget beyond that pool would block
        // the kernel at its first instruction, so the launch allocation is checked here, once, and never assumed
        cudaFuncAttributes fa;
        if (cudaFuncGetAttributes(&fa, kfn) != cudaSuccess) { delete m; return KG_E_CUDA; }
        if ((long long)fa.numRegs * DECODE_THREADS < (long long)NTHREADS * CONSUMER_REGS + 128LL * PRODUCER_REGS) {
            std::snprintf(g_cuda_err, sizeof(g_cuda_err), "decode kernel compiled with %d registers per thread: too few for its register budgets", fa.numRegs);
            delete m;
            return KG_E_INTERNAL;
        }
    }

    Dev& D = m->dev;
    std::memset(&D, 0, sizeof(D));
    D.dm.L = cfg->n_layers; D.dm.d = cfg->d_model; D.dm.H = cfg->n_heads; D.dm.hd = cfg->head_dim; D.dm.F = cfg->d_ffn;
    D.dm.V = cfg->vocab; D.dm.l = cfg->exit_layer; D.dm.eps = cfg->rms_eps; D.dm.theta = cfg->rope_theta;
    D.dm.logit_scale = cfg->logit_scale; D.dm.max_seq = cfg->max_seq; D.dm.page_size = cfg->page_size;
    D.dm.n_pages = (cfg->max_seq + cfg->page_size - 1) / cfg->page_size; D.dm.gamma_max = cfg->gamma_max;
    D.dm.n_phys = D.dm.n_pages;
    for (D.dm.ps_shift = 0; (1 << D.dm.ps_shift) < cfg->page_size; ++D.dm.ps_shift) {}
    D.dm.debug = cfg->debug_logits;
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        D.inv_freq[i] = std::pow((double)cfg->rope_theta, -2.0 * (double)i / (double)cfg->head_dim);
    auto P = [&](size_t off) { return base + off; };
    D.st = (State*)P(lay.off_st); D.bar = (unsigned*)P(lay.off_bar);
    D.layers = (const LayerW*)P(lay.off_layers); D.page_table = (const int*)P(lay.off_pt);
    D.kcache = P(lay.off_kc); D.vcache = P(lay.off_vc);
    D.h = (float*)P(lay.off_h); D.feat = (float*)P(lay.off_feat); D.abuf = (float*)P(lay.off_abuf);
    D.qkv = (float*)P(lay.off_qkv); D.attn = (float*)P(lay.off_attn); D.act = (float*)P(lay.off_act);
    D.att_po = (float*)P(lay.off_po); D.att_ml = (float*)P(lay.off_ml); D.att_cnt = (unsigned*)P(lay.off_cnt);
    D.head_part = (float4*)P(lay.off_hp);
    D.hA_pk = (unsigned char*)P(lay.off_hApk); D.hB_pk = (unsigned char*)P(lay.off_hBpk);
    D.attn_pk = (unsigned char*)P(lay.off_attnpk); D.act_pk = (unsigned char*)P(lay.off_actpk);
    D.featA_pk = (unsigned char*)P(lay.off_featApk); D.featD_pk = (unsigned char*)P(lay.off_featDpk);
    D.abuf_pk = (unsigned char*)P(lay.off_abufpk);
    D.ssq_hA = (float*)P(lay.off_ssqA); D.ssq_hB = (float*)P(lay.off_ssqB);
    D.ssq_feat = (float*)P(lay.off_ssqF); D.ssq_abuf = (float*)P(lay.off_ssqAb);
    D.dm.stream = (cfg->dtype == KG_BF16 && cfg->d_model % 16 == 0 && cfg->d_ffn % 16 == 0) ? 1 : 0;
    D.dbg_draft = cfg->debug_logits ? (float*)P(lay.off_dbgd) : nullptr;
    D.dbg_verify = cfg->debug_logits ? (float*)P(lay.off_dbgv) : nullptr;
    D.out_tokens = (int*)P(lay.off_out); D.S = (int*)P(lay.off_S); D.round_log = (int*)P(lay.off_rlog);
    D.prompt = (const int*)P(lay.off_prompt);

    const int nl = cfg->n_layers;
    m->layers_host.resize(nl + 1);
    if (own) {
        D.embed = P(lay.off_embed); D.head = P(lay.off_head); D.g_final = (const float*)P(lay.off_gfinal);
        for (int i = 0; i <= nl; ++i) {
            LayerW& lw = m->layers_host[i];
            lw.wqkv = P(lay.off_w[K_WQKV][i]); lw.wo = P(lay.off_w[K_WO][i]);
            lw.wgate = i < nl ? P(lay.off_w[K_WGATE][i]) : nullptr;
            lw.wup = i < nl ? P(lay.off_w[K_WUP][i]) : nullptr;
            lw.wdown = i < nl ? P(lay.off_w[K_WDOWN][i]) : nullptr;
            lw.g1 = (const float*)P(lay.off_g[0][i]); lw.g2 = (const float*)P(lay.off_g[1][i]);
        }
    } else {
        D.embed = w->embed_dev; D.head = w->head_dev; D.g_final = w->g_final_dev;
        for (int i = 0; i <= nl; ++i) {
            LayerW& lw = m->layers_host[i];
            lw.wqkv = w->wqkv_dev[i]; lw.wo = w->wo_dev[i];
            lw.wgate = i < nl ? w->wgate_dev[i] : nullptr;
            lw.wup = i < nl ? w->wup_dev[i] : nullptr;
            lw.wdown = i < nl ? w->wdown_dev[i] : nullptr;
            lw.g1 = w->g1_dev[i]; lw.g2 = w->g2_dev[i];
        }
    }
    cudaStream_t s = m->stream;
    bool ok = cudaMemcpyAsync(P(lay.off_layers), m->layers_host.data(), sizeof(LayerW) * (nl + 1), cudaMemcpyHostToDevice, s) == cudaSuccess;
    // page table: identity, or a fixed permutation (reversal within blocks of 4 pages plus a rotation)
    std::vector<int> pt(D.dm.n_pages);
    for (int i = 0; i < D.dm.n_pages; ++i) pt[i] = i;
    if (cfg->page_shuffle) {
        const int n = D.dm.n_pages;
        for (int i = 0; i < n; ++i) pt[i] = (int)(((long long)i * 7 + 3) % n);
        // i -> 7i+3 mod n is a permutation only if gcd(7, n) == 1; otherwise fall back to reversal
        if (n % 7 == 0) for (int i = 0; i < n; ++i) pt[i] = n - 1 - i;
    }
    ok = ok && cudaMemcpyAsync(P(lay.off_pt), pt.data(), sizeof(int) * pt.size(), cudaMemcpyHostToDevice, s) == cudaSuccess;
    ok = ok && cudaMemsetAsync(D.st, 0, sizeof(State), s) == cudaSuccess;
    ok = ok && cudaMemsetAsync(D.att_cnt, 0, 4 * cfg->n_heads, s) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;    // pt / layers_host are host temporaries
    if (!ok) { delete m; return KG_E_CUDA; }
    if (own) {
        int r = bf ? fill_weights<__nv_bfloat16>(m) : fill_weights<float>(m);
        // the fill kernels have run to completion (and without a fault) when the model is handed out
        if (r == KG_OK && cuda_failed(cudaStreamSynchronize(s), "weight fill")) r = KG_E_CUDA;
        if (r != KG_OK) { delete m; return r; }
    }
    *out = m;
    return KG_OK;
}

extern "C" int kg_free_model(kg_model* m) {
    if (!m) return KG_E_ARG;
    if (m->ev0) cudaEventDestroy(m->ev0);
    if (m->ev1) cudaEventDestroy(m->ev1);
    delete m;
    return KG_OK;
}

extern "C" int kg_reset(kg_model* m) {
    if (!m) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    CK(cudaMemsetAsync(m->dev.st, 0, sizeof(State), m->stream));
    CK(cudaMemsetAsync(m->dev.att_cnt, 0, 4 * m->cfg.n_heads, m->stream));
    m->prefilled = m->pending = m->ar_used = false;
    m->P_upper = 0;
    return KG_OK;
}

namespace {
int prefill_tc(kg_model* m, int n);                 // the tensor-core prompt pass (end of this file)
bool prefill_tc_ok(const kg_model* m, int n);
}

static int prefill_common(kg_model* m, int32_t n) {
    int r;
    if (prefill_tc_ok(m, n)) {
        r = prefill_tc(m, n);
    } else {
        Program pg{}; pg.kind = PROG_PREFILL; pg.n = n;
        r = launch(m, pg);
    }
    if (r != KG_OK) return r;
    m->prefilled = true; m->pending = false; m->P_upper = n;
    return KG_OK;
}

extern "C" int kg_prefill(kg_model* m, const int32_t* prompt_host, int32_t n, int32_t* first_token_host) {
    if (!m || !prompt_host || n < 1) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (m->prefilled || m->ar_used) return KG_E_STATE;
    if (n + 1 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    for (int i = 0; i < n; ++i) if (prompt_host[i] < 0 || prompt_host[i] >= m->cfg.vocab) return KG_E_ARG;
    CK(cudaMemcpyAsync((void*)m->dev.prompt, prompt_host, sizeof(int32_t) * n, cudaMemcpyHostToDevice, m->stream));
    int r = prefill_common(m, n);
    if (r != KG_OK) return r;
    if (first_token_host) {
        State st;
        r = read_state(m, &st);
        if (r != KG_OK) return r;
        *first_token_host = st.x0;
    } else {
        // the prompt buffer is the caller's: make sure the copy has left it
        CK(cudaStreamSynchronize(m->stream));
    }
    return KG_OK;
}

extern "C" int kg_prefill_device(kg_model* m, const int32_t* prompt_dev, int32_t n) {
    if (!m || !prompt_dev || n < 1) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (m->prefilled || m->ar_used) return KG_E_STATE;
    if (n + 1 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    if (reinterpret_cast<uintptr_t>(prompt_dev) & 3u) return KG_E_ARG;
    CK(cudaMemcpyAsync((void*)m->dev.prompt, prompt_dev, sizeof(int32_t) * n, cudaMemcpyDeviceToDevice, m->stream));
    check_tokens_kernel<<<(n + 255) / 256, 256, 0, m->stream>>>(m->dev.prompt, n, m->cfg.vocab, m->dev.st);
    CK(cudaGetLastError());
    return prefill_common(m, n);
}

static bool bad_spec(const kg_model* m, float eta, int gamma, int mode) {
    return !(eta == eta) || gamma < 1 || gamma > m->cfg.gamma_max || (mode != KG_STOP_KEEP && mode != KG_STOP_DROP);
}

extern "C" int kg_draft(kg_model* m, float eta, int32_t gamma, int32_t stop_mode, kg_draft_out* out) {
    if (!m || bad_spec(m, eta, gamma, stop_mode)) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (!m->prefilled || m->pending || m->ar_used) return KG_E_STATE;
    if (m->P_upper + gamma + 2 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    Program pg{}; pg.kind = PROG_DRAFT; pg.eta = eta; pg.gamma = gamma; pg.stop_mode = stop_mode;
    int r = launch(m, pg);
    if (r != KG_OK) return r;
    m->pending = true; m->gamma_pending = gamma;
    if (out) {
        State st;
        r = read_state(m, &st);
        if (r != KG_OK) return r;
        out->n_drafted = st.n_d; out->n_steps = st.n_steps;
        for (int i = 0; i < KG_GAMMA_MAX; ++i) { out->tokens[i] = i < st.n_d ? st.draft_tok[i] : -1; out->conf[i] = i < st.n_steps ? st.conf[i] : 0.f; }
    }
    return KG_OK;
}

extern "C" int kg_verify(kg_model* m, kg_verify_out* out) {
    if (!m) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (!m->prefilled || !m->pending) return KG_E_STATE;
    Program pg{}; pg.kind = PROG_VERIFY;
    int r = launch(m, pg);
    if (r != KG_OK) return r;
    m->pending = false;
    m->P_upper += m->gamma_pending + 1;
    if (out) {
        State st;
        r = read_state(m, &st);
        if (r != KG_OK) return r;
        out->n_rows = st.M; out->n_accept = st.k_acc; out->n_emitted = st.n_emit;
        for (int i = 0; i < KG_M_MAX; ++i) { out->emitted[i] = i < st.n_emit ? st.emitted[i] : -1; out->target[i] = i < st.M ? st.target[i] : -1; }
        m->P_upper = st.P;
    }
    return KG_OK;
}

static void fill_stats(kg_model* m, const State& st, const std::vector<int>& S, int max_tokens, kg_stats* out) {
    std::memset(out, 0, sizeof(*out));
    std::vector<int> s2(S);
    // truncate so that only tokens up to max_tokens (x_0 excluded from S) are counted
    long long sum = 0;
    for (size_t i = 0; i < s2.size(); ++i) {
        if (max_tokens >= 0 && sum + s2[i] > max_tokens - 1) { s2[i] = (int)(max_tokens - 1 - sum); s2.resize(s2[i] > 0 ? i + 1 : i); sum = max_tokens - 1; break; }
        sum += s2[i];
    }
    out->rounds = (int)s2.size(); out->tokens = (int)sum;
    out->draft_steps = st.draft_steps_total; out->drafted = st.drafted_total; out->accepted = st.accepted_total;
    if (!s2.empty()) {
        out->cr = (double)sum / (double)s2.size();
        for (int w = 0; w <= KG_M_MAX; ++w) {
            int cnt = 0;
            for (int v : s2) cnt += (v - w > 0);
            out->ctar[w] = (double)cnt / (double)s2.size();
        }
    }
}

static int read_S_vec(kg_model* m, int rounds, std::vector<int>& S) {
    S.assign(rounds, 0);
    if (rounds > 0) {
        CK(cudaMemcpyAsync(S.data(), m->dev.S, sizeof(int) * rounds, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    return KG_OK;
}

extern "C" int kg_decode(kg_model* m, int32_t max_new, float eta, int32_t gamma, int32_t stop_mode, kg_stats* stats) {
    if (!m || bad_spec(m, eta, gamma, stop_mode) || max_new < 1) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (!m->prefilled || m->pending || m->ar_used) return KG_E_STATE;
    if (m->P_upper + max_new + gamma + 2 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    Program pg{}; pg.kind = PROG_DECODE; pg.n = max_new; pg.eta = eta; pg.gamma = gamma; pg.stop_mode = stop_mode;
    int r = launch(m, pg);
    if (r != KG_OK) return r;
    m->P_upper += max_new + gamma + 1;
    if (stats) {
        State st;
        r = read_state(m, &st);
        if (r != KG_OK) return r;
        m->P_upper = st.P;
        std::vector<int> S;
        r = read_S_vec(m, st.rounds, S);
        if (r != KG_OK) return r;
        fill_stats(m, st, S, max_new, stats);
    }
    return KG_OK;
}

extern "C" int kg_decode_ar(kg_model* m, int32_t n_tokens, int32_t* out_host) {
    if (!m || n_tokens < 1) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    if (!m->prefilled || m->pending) return KG_E_STATE;
    if (m->P_upper + n_tokens + 1 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    Program pg{}; pg.kind = PROG_AR; pg.n = n_tokens;
    int r = launch(m, pg);
    if (r != KG_OK) return r;
    m->ar_used = true;
    m->P_upper += n_tokens;
    if (out_host) {
        State st;
        r = read_state(m, &st);
        if (r != KG_OK) return r;
        CK(cudaMemcpyAsync(out_host, m->dev.out_tokens, sizeof(int) * n_tokens, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    return KG_OK;
}

extern "C" int kg_read_tokens(kg_model* m, int32_t* out_host, int32_t max_n, int32_t* n_out) {
    if (!m || !out_host || max_n < 0) return KG_E_ARG;
    State st;
    int r = read_state(m, &st);
    if (r != KG_OK) return r;
    const int n = st.total < max_n ? st.total : max_n;
    if (n > 0) {
        CK(cudaMemcpyAsync(out_host, m->dev.out_tokens, sizeof(int) * n, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    if (n_out) *n_out = n;
    return KG_OK;
}

extern "C" int kg_read_S(kg_model* m, int32_t* out_host, int32_t max_n, int32_t* n_out) {
    if (!m || !out_host || max_n < 0) return KG_E_ARG;
    State st;
    int r = read_state(m, &st);
    if (r != KG_OK) return r;
    const int n = st.rounds < max_n ? st.rounds : max_n;
    if (n > 0) {
        CK(cudaMemcpyAsync(out_host, m->dev.S, sizeof(int) * n, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    if (n_out) *n_out = n;
    return KG_OK;
}

extern "C" int kg_read_round_log(kg_model* m, int32_t* out_host, int32_t max_rounds, int32_t* n_out) {
    if (!m || !out_host || max_rounds < 0) return KG_E_ARG;
    State st;
    int r = read_state(m, &st);
    if (r != KG_OK) return r;
    const int n = st.rounds < max_rounds ? st.rounds : max_rounds;
    if (n > 0) {
        CK(cudaMemcpyAsync(out_host, m->dev.round_log, sizeof(int) * 4 * n, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    }
    if (n_out) *n_out = n;
    return KG_OK;
}

extern "C" int kg_generate(kg_model* m, const int32_t* prompt_host, int32_t n_prompt, int32_t max_new,
                           float eta, int32_t gamma, int32_t stop_mode,
                           int32_t* out_tokens_host, int32_t* n_out, kg_stats* stats) {
    if (!m || !prompt_host || !out_tokens_host || max_new < 1 || bad_spec(m, eta, gamma, stop_mode)) return KG_E_ARG;
    if ((long long)n_prompt + max_new + gamma + 2 > m->cfg.max_seq) return KG_E_SEQ_FULL;
    int r = kg_reset(m);
    if (r != KG_OK) return r;
    for (int i = 0; i < n_prompt; ++i) if (prompt_host[i] < 0 || prompt_host[i] >= m->cfg.vocab) return KG_E_ARG;
    if (n_prompt < 1) return KG_E_ARG;
    CK(cudaMemcpyAsync((void*)m->dev.prompt, prompt_host, sizeof(int32_t) * n_prompt, cudaMemcpyHostToDevice, m->stream));
    r = prefill_common(m, n_prompt);
    if (r != KG_OK) return r;
    const bool timed = stats != nullptr;
    if (timed) {
        if (!m->ev0) { CK(cudaEventCreate(&m->ev0)); CK(cudaEventCreate(&m->ev1)); }      // once per model
        CK(cudaEventRecord(m->ev0, m->stream));
    }
    r = kg_decode(m, max_new, eta, gamma, stop_mode, nullptr);
    if (timed && r == KG_OK) cudaEventRecord(m->ev1, m->stream);
    State st;
    if (r == KG_OK) r = read_state(m, &st);
    if (r == KG_OK) {
        if (cudaMemcpyAsync(out_tokens_host, m->dev.out_tokens, sizeof(int) * max_new, cudaMemcpyDeviceToHost, m->stream) != cudaSuccess ||
            cudaStreamSynchronize(m->stream) != cudaSuccess) r = KG_E_CUDA;
    }
    if (r == KG_OK) {
        m->P_upper = st.P;
        if (n_out) *n_out = max_new;
        if (stats) {
            std::vector<int> S;
            r = read_S_vec(m, st.rounds, S);
            if (r == KG_OK) {
                fill_stats(m, st, S, max_new, stats);
                float ms = 0.f;
                if (cudaEventElapsedTime(&ms, m->ev0, m->ev1) == cudaSuccess) stats->ms_decode = ms;
            }
        }
    }
    return r;
}

extern "C" int kg_debug_logits(kg_model* m, int32_t which, int32_t row, float* out_host) {
    if (!m || !out_host || row < 0 || row >= KG_M_MAX || (which != 0 && which != 1)) return KG_E_ARG;
    if (!m->cfg.debug_logits) return KG_E_STATE;
    const float* src = (which == 0 ? m->dev.dbg_draft : m->dev.dbg_verify) + (size_t)row * m->cfg.vocab;
    CK(cudaMemcpyAsync(out_host, src, sizeof(float) * m->cfg.vocab, cudaMemcpyDeviceToHost, m->stream));
    CK(cudaStreamSynchronize(m->stream));
    return KG_OK;
}

extern "C" int kg_read_weight(kg_model* m, const char* name, int32_t layer, uint64_t offset, uint64_t count, float* out_host) {
    if (!m || !name || !out_host) return KG_E_ARG;
    const kg_config& c = m->cfg;
    const uint64_t d = c.d_model, F = c.d_ffn, V = c.vocab;
    const void* p = nullptr; uint64_t n = 0; bool f32 = false;
    const bool lay_ok = layer >= 0 && layer <= c.n_layers;
    if (!std::strcmp(name, "embed")) { p = m->dev.embed; n = V * d; }
    else if (!std::strcmp(name, "head")) { p = m->dev.head; n = V * d; }
    else if (!std::strcmp(name, "g_final")) { p = m->dev.g_final; n = d; f32 = true; }
    else if (!lay_ok) return KG_E_ARG;
    else if (!std::strcmp(name, "wqkv")) { p = m->layers_host[layer].wqkv; n = 3 * d * d; }
    else if (!std::strcmp(name, "wo")) { p = m->layers_host[layer].wo; n = d * d; }
    else if (!std::strcmp(name, "wgate")) { p = m->layers_host[layer].wgate; n = F * d; }
    else if (!std::strcmp(name, "wup")) { p = m->layers_host[layer].wup; n = F * d; }
    else if (!std::strcmp(name, "wdown")) { p = m->layers_host[layer].wdown; n = d * F; }
    else if (!std::strcmp(name, "g1")) { p = m->layers_host[layer].g1; n = d; f32 = true; }
    else if (!std::strcmp(name, "g2")) { p = m->layers_host[layer].g2; n = d; f32 = true; }
    else return KG_E_ARG;
    if (!p || offset > n || count > n - offset) return KG_E_ARG;
    if (f32 || c.dtype == KG_F32) {
        CK(cudaMemcpyAsync(out_host, (const float*)p + offset, 4 * count, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
    } else {
        std::vector<uint16_t> tmp(count);
        CK(cudaMemcpyAsync(tmp.data(), (const uint16_t*)p + offset, 2 * count, cudaMemcpyDeviceToHost, m->stream));
        CK(cudaStreamSynchronize(m->stream));
        for (uint64_t i = 0; i < count; ++i) { uint32_t b = (uint32_t)tmp[i] << 16; std::memcpy(out_host + i, &b, 4); }
    }
    return KG_OK;
}

extern "C" int kg_debug_fill_state(kg_model* m, int32_t T, int32_t n_d, uint64_t seed) {
    if (!m || T < 1 || n_d < -1 || n_d > m->cfg.gamma_max) return KG_E_ARG;
    if (m->dead) return KG_E_TIMEOUT;
    const kg_config& c = m->cfg;
    if (T + c.gamma_max + 2 > c.max_seq) return KG_E_SEQ_FULL;
    cudaStream_t s = m->stream;
    const float one = gen_scale(1.0);
    const size_t lstride = (size_t)m->dev.dm.n_pages * c.n_heads * c.page_size * c.head_dim;
    for (int i = 0; i <= c.n_layers; ++i) {
        if (c.dtype == KG_BF16) {
            fill_cache_kernel<__nv_bfloat16><<<592, 256, 0, s>>>((__nv_bfloat16*)m->dev.kcache + i * lstride, m->dev.page_table, stream_base(seed, layer_tid(i, K_KCACHE)), T, c.n_heads, c.head_dim, c.page_size, one);
            fill_cache_kernel<__nv_bfloat16><<<592, 256, 0, s>>>((__nv_bfloat16*)m->dev.vcache + i * lstride, m->dev.page_table, stream_base(seed, layer_tid(i, K_VCACHE)), T, c.n_heads, c.head_dim, c.page_size, one);
        } else {
            fill_cache_kernel<float><<<592, 256, 0, s>>>((float*)m->dev.kcache + i * lstride, m->dev.page_table, stream_base(seed, layer_tid(i, K_KCACHE)), T, c.n_heads, c.head_dim, c.page_size, one);
            fill_cache_kernel<float><<<592, 256, 0, s>>>((float*)m->dev.vcache + i * lstride, m->dev.page_table, stream_base(seed, layer_tid(i, K_VCACHE)), T, c.n_heads, c.head_dim, c.page_size, one);
        }
    }
    fill_f32_kernel<<<64, 256, 0, s>>>(m->dev.feat, stream_base(seed, TID_HIDDEN), (uint64_t)(KG_M_MAX + 1) * c.d_model, one);
    if (m->dev.dm.stream) {
        const int d = c.d_model;
        pack_rows_kernel<<<m->nctas, 256, 0, s>>>(m->dev.feat, d, KG_M_MAX + 1, d, m->layers_host[c.n_layers].g1, m->dev.featA_pk, d * 4, m->dev.ssq_feat, m->nctas);
        pack_rows_kernel<<<m->nctas, 256, 0, s>>>(m->dev.feat, d, KG_M_MAX + 1, d, m->layers_host[c.exit_layer].g1, m->dev.featD_pk, d * 4, m->dev.ssq_feat, m->nctas);
    }
    CK(cudaGetLastError());
    // tokens: x_0 and the drafts
    const uint64_t tb = stream_base(seed, TID_DRAFT);
    State st;
    std::memset(&st, 0, sizeof(st));
    st.P = T; st.len_A = T; st.total = 1; st.x0 = (int)(mix64(tb + 1000) % (uint64_t)c.vocab);
    if (n_d >= 0) {
        st.pending = 1; st.n_d = n_d; st.n_steps = n_d;
        for (int i = 0; i < n_d; ++i) { st.draft_tok[i] = (int)(mix64(tb + (uint64_t)i) % (uint64_t)c.vocab); st.conf[i] = 1.0f; }
    }
    CK(cudaMemcpyAsync(m->dev.st, &st, sizeof(State), cudaMemcpyHostToDevice, s));
    CK(cudaMemsetAsync(m->dev.att_cnt, 0, 4 * c.n_heads, s));
    CK(cudaStreamSynchronize(s));
    m->prefilled = true; m->pending = n_d >= 0; m->ar_used = false; m->gamma_pending = n_d >= 0 ? n_d : 0; m->P_upper = T;
    return KG_OK;
}

extern "C" int kg_debug_force_simple(kg_model* m, int on) {
    if (!m) return KG_E_ARG;
    // the plain path stages all rows of an operand in shared memory: only shapes whose rows fit may take it
    const int kmax = m->cfg.d_ffn > m->cfg.d_model ? m->cfg.d_ffn : m->cfg.d_model;
    if (on && (size_t)kmax * KG_M_MAX * 4 > (size_t)SIMPLE_XS_BYTES) return KG_E_ARG;
    m->force_simple = on ? 1 : 0;
    return KG_OK;
}

extern "C" int kg_debug_set_wait_budget(kg_model* m, double milliseconds) {
    if (!m || !(milliseconds > 0.0) || milliseconds > 60000.0) return KG_E_ARG;
    int dev = 0, khz = 0;
    CK(cudaGetDevice(&dev));
    CK(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
    m->wait_clk = (unsigned long long)(milliseconds * (double)khz);      // kHz = clocks per millisecond
    if (m->wait_clk < 1000ull) m->wait_clk = 1000ull;
    return KG_OK;
}

extern "C" int kg_debug_skip_barrier_arrival(kg_model* m, int cta) {
    if (!m || cta < 0 || cta >= m->nctas) return KG_E_ARG;
    m->skip_arrival = cta + 1;
    return KG_OK;
}

// ------------------------------------------------------------------------------------ single operators
namespace {

constexpr int OP_K_MAX = 32768;               // longest input row the single-operator entry points pack into scratch
struct OpScratch { size_t off_hp, off_po, off_ml, off_cnt, off_pt, off_xpk, off_ssq, total; };
OpScratch op_layout() {
    OpScratch s; size_t o = 0;
    auto take = [&](size_t b) { size_t r = o; o = align_up(o + b, 256); return r; };
    s.off_hp = take(sizeof(float4) * 1024 * KG_M_MAX);
    s.off_po = take(4 * (size_t)KG_M_MAX * S_CAP * 8192);
    s.off_ml = take(4 * (size_t)KG_M_MAX * 256 * S_CAP * 2);
    s.off_cnt = take(4 * 256);
    s.off_xpk = take(4 * (size_t)KG_M_MAX * OP_K_MAX);
    s.off_ssq = take(4 * (size_t)KG_M_MAX * 1024);
    s.total = o;
    return s;
}

template <typename WT>
__global__ void __launch_bounds__(BLOCK_THREADS, 1) op_linear_kernel(LinArgs a, int stream) {
    extern __shared__ __align__(128) char smem[];
    Ctx& c = ctx_init(smem, nullptr, nullptr, false);
    OpTable* t = reinterpret_cast<OpTable*>(c.producer ? c.ctl->tab_prod : c.ctl->tab_cons);
    if (c.producer ? (threadIdx.x & 31) == 0 : threadIdx.x == 0) t->lin[0] = a;
    const bool ok = linear_op<WT>(&t->lin[0], c, stream != 0, true);
    if (!ok && c.producer) ring_drain(c);
}
__global__ void op_head_final_kernel(const float4* part, int nctas, int M, int* tok, float* p) {
    if (threadIdx.x < M) { int t; float pp; head_final(part, nctas, threadIdx.x, t, pp); tok[threadIdx.x] = t; p[threadIdx.x] = pp; }
}
template <typename WT>
__global__ void __launch_bounds__(BLOCK_THREADS, 1) op_attention_kernel(const __grid_constant__ Dev D, AttArgs a) {
    extern __shared__ __align__(128) char smem[];
    Ctx& c = ctx_init(smem, nullptr, nullptr, false);
    if (!c.producer) {
        OpTable* t = reinterpret_cast<OpTable*>(c.ctl->tab_cons);
        if (threadIdx.x == 0) t->att = a;
        cta_sync();
        attention_op<WT>(D, &t->att, c);
    }
}

int g_force_simple_ops = 0;

template <typename K>
int set_smem(K kfn) {
    return cudaFuncSetAttribute((const void*)kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_TOTAL) == cudaSuccess ? KG_OK : KG_E_CUDA;
}

}  // namespace

extern "C" size_t kg_op_scratch_bytes(void) { return op_layout().total; }

extern "C" int kg_debug_force_simple_ops(int on) { g_force_simple_ops = on ? 1 : 0; return KG_OK; }

// xpk / ssq: scratch for the packed copy of the input rows (xpk_k_max = longest row it holds) and their sums of squares
static int op_linear_common(int32_t dtype, LinArgs& a, unsigned char* xpk, int xpk_k_max, float* ssq, cudaStream_t s) {
    if (dtype != KG_F32 && dtype != KG_BF16) return KG_E_ARG;
    if (a.M < 1 || a.M > KG_M_MAX || a.N < 1 || a.N > (1 << 20) || a.K < 8 || (a.K % 8)) return KG_E_ARG;
    const bool plain = dtype == KG_F32 || g_force_simple_ops || (a.K % 16);
    if (plain && (size_t)a.K * a.M * 4 > (size_t)SIMPLE_XS_BYTES) return KG_E_ARG;
    const int nctas = sm_count();
    if (!plain) {
        if (a.K > xpk_k_max || nctas > 1024) return KG_E_LIMIT;
        pack_rows_kernel<<<nctas, 256, 0, s>>>(a.x, a.ldx, a.M, a.K, a.gain, xpk, a.K * 4, a.gain ? ssq : nullptr, nctas);
        a.xpk = xpk; a.ldpk = a.K * 4; a.ssq_in = a.gain ? ssq : nullptr;
    }
    if (dtype == KG_BF16) {
        if (set_smem(op_linear_kernel<__nv_bfloat16>) != KG_OK) return KG_E_CUDA;
        op_linear_kernel<__nv_bfloat16><<<nctas, BLOCK_THREADS, SMEM_TOTAL, s>>>(a, plain ? 0 : 1);
    } else {
        if (set_smem(op_linear_kernel<float>) != KG_OK) return KG_E_CUDA;
        op_linear_kernel<float><<<nctas, BLOCK_THREADS, SMEM_TOTAL, s>>>(a, 0);
    }
    CK(cudaGetLastError());
    return KG_OK;
}

extern "C" int kg_op_linear(int32_t dtype, const void* W, const void* W2, int32_t N, int32_t K,
                            const float* x, int32_t M, const float* gain, float eps,
                            const float* resid, int32_t swiglu, float* out, void* scratch, void* stream) {
    if (!W || !x || !out || !scratch) return KG_E_ARG;
    if (swiglu && !W2) return KG_E_ARG;
    if (!aligned16(W) || !aligned16(W2) || !aligned16(x) || !aligned16(gain) || !aligned16(resid) || !aligned16(out) ||
        !aligned16(scratch)) return KG_E_ARG;
    LinArgs a{};
    a.W = W; a.W2 = swiglu ? W2 : nullptr; a.N = N; a.K = K; a.x = x; a.ldx = K; a.M = M; a.gain = gain; a.eps = eps;
    a.resid = resid; a.ldr = N; a.out = out; a.ldo = N;
    a.epi = swiglu ? EPI_SWIGLU : (resid ? EPI_RESID : EPI_STORE);
    OpScratch sc = op_layout();
    return op_linear_common(dtype, a, (unsigned char*)scratch + sc.off_xpk, OP_K_MAX, (float*)((char*)scratch + sc.off_ssq), (cudaStream_t)stream);
}

extern "C" int kg_op_lm_head(int32_t dtype, const void* W, int32_t V, int32_t K, const float* x, int32_t M,
                             const float* gain, float eps, float logit_scale,
                             int32_t* tok, float* p, float* logits, void* scratch, void* stream) {
    if (!W || !x || !tok || !p || !scratch) return KG_E_ARG;
    if (!aligned16(W) || !aligned16(x) || !aligned16(gain) || !aligned16(logits) || !aligned16(scratch) ||
        (reinterpret_cast<uintptr_t>(tok) & 3u) || (reinterpret_cast<uintptr_t>(p) & 3u)) return KG_E_ARG;
    if (sm_count() > 1024) return KG_E_ARG;
    OpScratch sc = op_layout();
    LinArgs a{};
    a.W = W; a.N = V; a.K = K; a.x = x; a.ldx = K; a.M = M; a.gain = gain; a.eps = eps;
    a.epi = EPI_HEAD; a.scale = logit_scale; a.head_part = (float4*)((char*)scratch + sc.off_hp);
    a.logits_dbg = logits; a.ld_dbg = V;
    int r = op_linear_common(dtype, a, (unsigned char*)scratch + sc.off_xpk, OP_K_MAX, (float*)((char*)scratch + sc.off_ssq), (cudaStream_t)stream);
    if (r != KG_OK) return r;
    op_head_final_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(a.head_part, sm_count(), M, tok, p);
    CK(cudaGetLastError());
    return KG_OK;
}

// ------------------------------------------------------------------------------------ no-allocation variant
// The LM-head operator keeps one partial (max, sum, arg max) per CTA and row in scratch memory.  Here that
// scratch is a fixed array inside the library image instead of caller memory.
namespace {
constexpr int NOALLOC_MAX_CTAS = 256;                        // CTAs (one per SM) the static scratch has room for
constexpr int NOALLOC_MAX_K = 8192;                          // longest input row it can pack
constexpr int NOALLOC_MAX_DEVICES = 64;
constexpr size_t NOALLOC_OFF_XPK = sizeof(float4) * NOALLOC_MAX_CTAS * KG_M_MAX;                 // head partials first: 64 KB
constexpr size_t NOALLOC_OFF_SSQ = NOALLOC_OFF_XPK + 4 * (size_t)KG_M_MAX * NOALLOC_MAX_K;        // packed input rows: 512 KB
constexpr size_t NOALLOC_BYTES = NOALLOC_OFF_SSQ + 4 * (size_t)KG_M_MAX * NOALLOC_MAX_CTAS;       // sums of squares: 16 KB
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];
static_assert(NOALLOC_MAX_DEVICES <= MAX_DEVICES, "per-device tables");
void* g_noalloc_addr[NOALLOC_MAX_DEVICES] = {nullptr};

// Device address of the static scratch on the current device.  In host code the array's name is only a
// handle for the runtime, never a pointer a kernel may use; the address comes from cudaGetSymbolAddress.
int noalloc_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return KG_E_CUDA;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return KG_E_LIMIT;
    if (!g_noalloc_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return KG_E_CUDA;
        g_noalloc_addr[dev] = p;
    }
    *out = g_noalloc_addr[dev];
    return KG_OK;
}
}  // namespace

extern "C" int kg_op_lm_head_noalloc(int32_t dtype, const void* W, int32_t V, int32_t K, const float* x, int32_t M,
                                     const float* gain, float eps, float logit_scale,
                                     int32_t* tok, float* p, float* logits, void* stream) {
    if (!W || !x || !tok || !p) return KG_E_ARG;
    if (!aligned16(W) || !aligned16(x) || !aligned16(gain) || !aligned16(logits) ||
        (reinterpret_cast<uintptr_t>(tok) & 3u) || (reinterpret_cast<uintptr_t>(p) & 3u)) return KG_E_ARG;
    if (M > KG_M_MAX || K > NOALLOC_MAX_K || sm_count() > NOALLOC_MAX_CTAS) return KG_E_LIMIT;
    void* scratch = nullptr;
    int r = noalloc_scratch(&scratch);
    if (r != KG_OK) return r;
    // the partials of an earlier call are stale but harmless: every CTA rewrites its rows before they are merged
    LinArgs a{};
    a.W = W; a.N = V; a.K = K; a.x = x; a.ldx = K; a.M = M; a.gain = gain; a.eps = eps;
    a.epi = EPI_HEAD; a.scale = logit_scale; a.head_part = (float4*)scratch;
    a.logits_dbg = logits; a.ld_dbg = V;
    r = op_linear_common(dtype, a, (unsigned char*)scratch + NOALLOC_OFF_XPK, NOALLOC_MAX_K, (float*)((char*)scratch + NOALLOC_OFF_SSQ),
                         (cudaStream_t)stream);
    if (r != KG_OK) return r;
    op_head_final_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(a.head_part, sm_count(), M, tok, p);
    CK(cudaGetLastError());
    return KG_OK;
}

extern "C" int kg_op_attention(int32_t dtype, const float* qkv, int32_t M, int32_t pos0, int32_t H, int32_t hd,
                               float theta, void* kc, void* vc, const int32_t* page_table, int32_t page_size,
                               float* out, void* scratch, void* stream) {
    if (!qkv || !kc || !vc || !page_table || !out || !scratch) return KG_E_ARG;
    if (dtype != KG_F32 && dtype != KG_BF16) return KG_E_ARG;
    if (!aligned16(qkv) || !aligned16(kc) || !aligned16(vc) || !aligned16(out) || !aligned16(scratch) ||
        (reinterpret_cast<uintptr_t>(page_table) & 3u)) return KG_E_ARG;
    if (M < 1 || M > KG_M_MAX || pos0 < 0 || H < 1 || H > 256 || (hd != 32 && hd != 64 && hd != 128) || page_size < 1 ||
        (page_size & (page_size - 1))) return KG_E_ARG;
    if ((size_t)H * hd > 8192) return KG_E_ARG;
    OpScratch sc = op_layout();
    cudaStream_t s = (cudaStream_t)stream;
    Dev D;
    std::memset(&D, 0, sizeof(D));
    D.dm.H = H; D.dm.hd = hd; D.dm.d = H * hd; D.dm.page_size = page_size; D.dm.theta = theta;
    D.dm.n_pages = (pos0 + M + page_size - 1) / page_size;       // entries of page_table this call may touch
    D.dm.n_phys = 0x7fffffff;                                    // the caller's cache: its page count is not known here
    for (D.dm.ps_shift = 0; (1 << D.dm.ps_shift) < page_size; ++D.dm.ps_shift) {}
    for (int i = 0; i < hd / 2; ++i) D.inv_freq[i] = std::pow((double)theta, -2.0 * (double)i / (double)hd);
    D.page_table = page_table;
    D.att_po = (float*)((char*)scratch + sc.off_po); D.att_ml = (float*)((char*)scratch + sc.off_ml);
    D.att_cnt = (unsigned*)((char*)scratch + sc.off_cnt);
    CK(cudaMemsetAsync(D.att_cnt, 0, 4 * 256, s));
    AttArgs a; a.qkv = qkv; a.M = M; a.pos0 = pos0; a.kc = kc; a.vc = vc; a.out = out;
    const int nctas = sm_count();
    if (dtype == KG_BF16) {
        if (set_smem(op_attention_kernel<__nv_bfloat16>) != KG_OK) return KG_E_CUDA;
        op_attention_kernel<__nv_bfloat16><<<nctas, BLOCK_THREADS, SMEM_TOTAL, s>>>(D, a);
    } else {
        if (set_smem(op_attention_kernel<float>) != KG_OK) return KG_E_CUDA;
        op_attention_kernel<float><<<nctas, BLOCK_THREADS, SMEM_TOTAL, s>>>(D, a);
    }
    CK(cudaGetLastError());
    return KG_OK;
}

// ------------------------------------------------------------------------------------ tensor-core prompt pass
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled of the driver, looked up through the runtime (the library does not link libcuda)
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map of a row-major bf16 matrix [rows, K] read in boxes of 64 columns x 128 rows with the 128-byte swizzle.
// base is 16-byte aligned and K * 2 a multiple of 16 (checked by the callers' shape test).
bool make_tmap(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)GM_BK, (cuuint32_t)GM_BM};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// launched with the consumer warps only (no copy warp: nothing is streamed), which leaves 255 registers per thread
__global__ void __launch_bounds__(NTHREADS, 1) pf_attention_kernel(const __grid_constant__ Dev D, AttArgs a, int nrows) {
    extern __shared__ __align__(128) char smem[];
    Ctx& c = ctx_init(smem, nullptr, nullptr, false);
    if (D.dm.hd == 128) attention_prefill<128>(D, a, c, nrows);
    else attention_prefill<64>(D, a, c, nrows);
}

// x_0 from the per-CTA LM-head partials; the sequence state after a prompt of n tokens (one warp)
__global__ void pf_finish_kernel(const float4* part, int nctas, State* st, int* out_tokens, int n, const int* gemm_err) {
    int tok; float p;
    head_final_warp(part, nctas, 0, tok, p);
    if (threadIdx.x == 0) {
        if (*gemm_err) { atomicCAS(&st->status, 0, ST_TIMEOUT); st->timeout_where = 60; }      // a wait inside a GEMM gave up
        st->P = n; st->len_A = n; st->x0 = tok; st->pending = 0; st->total = 1; st->rounds = 0;
        out_tokens[0] = tok;
    }
}

bool prefill_tc_ok(const kg_model* m, int n) {
    return m->prefill_mode == 0 && m->dev.dm.stream != 0 && prefill_tc_shape(&m->cfg) && n >= 2 * KG_M_MAX && encode_tiled_fn() != nullptr;
}

// C[rows, N] = (resid) + rowscale * planes[rows, K] W[N, K]^T; with W2: also C2 = rowscale * planes W2^T in the same launch
int pf_gemm(kg_model* m, const void* W, int N, int K, int rows, float* C, const float* resid, const float* rowscale,
            const void* W2 = nullptr, float* C2 = nullptr) {
    char* A = m->arena;
    const int rows_pad = (rows + GM_BM - 1) / GM_BM * GM_BM;
    CUtensorMap th, tl, tw, tw2;
    if (!make_tmap(&th, A + m->lay.off_pf_hi, rows_pad, K) || !make_tmap(&tl, A + m->lay.off_pf_lo, rows_pad, K) || !make_tmap(&tw, W, N, K) ||
        !make_tmap(&tw2, W2 ? W2 : W, N, K)) {
        std::snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed");
        return KG_E_CUDA;
    }
    GemmArgs g;
    g.C = C; g.C2 = C2; g.ldc = N; g.resid = resid; g.ldr = N; g.rowscale = rowscale; g.rows = rows; g.N = N; g.K = K; g.err = (int*)(A + m->lay.off_pf_err);
    pf_gemm_kernel<<<dim3(N / GM_BN, rows_pad / GM_BM, W2 ? 2 : 1), GM_THREADS, GM_SMEM, m->stream>>>(th, tl, tw, tw2, g);
    CK(cudaGetLastError());
    return KG_OK;
}

// The prompt in blocks of PF_ROWS rows, each block through all layers (its K / V are in the caches before the next
// block attends to them), the adapter's K / V after layer l, the LM head on the last row.
int prefill_tc(kg_model* m, int n) {
    typedef __nv_bfloat16 WT;
    const kg_config& c = m->cfg;
    const Dev& D = m->dev;
    cudaStream_t s = m->stream;
    char* A = m->arena;
    const int d = c.d_model, F = c.d_ffn, L = c.n_layers, H = c.n_heads;
    float* h = (float*)(A + m->lay.off_pf_h); float* h2 = (float*)(A + m->lay.off_pf_h2);
    float* qkv = (float*)(A + m->lay.off_pf_qkv); float* attn = (float*)(A + m->lay.off_pf_attn);
    float* gate = (float*)(A + m->lay.off_pf_gate); float* up = (float*)(A + m->lay.off_pf_up);
    WT* hi = (WT*)(A + m->lay.off_pf_hi); WT* lo = (WT*)(A + m->lay.off_pf_lo);
    float* rs = (float*)(A + m->lay.off_pf_err) + 16;               // [PF_ROWS] 1/rms of the rows the planes were made from
    CK(cudaFuncSetAttribute((const void*)pf_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM));
    CK(cudaFuncSetAttribute((const void*)pf_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_TOTAL));
    CK(cudaFuncSetAttribute((const void*)op_linear_kernel<WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_TOTAL));
    CK(cudaMemsetAsync(A + m->lay.off_pf_err, 0, 4, s));
    const size_t lstride = (size_t)D.dm.n_pages * H * c.page_size * c.head_dim;
    int r = KG_OK;
    for (int b0 = 0; b0 < n; b0 += PF_ROWS) {
        const int rows = n - b0 < PF_ROWS ? n - b0 : PF_ROWS;
        pf_embed_kernel<WT><<<rows, 256, 0, s>>>(D.prompt + b0, (const WT*)D.embed, c.vocab, d, h);
        auto qkv_and_append = [&](const LayerW& lw, int li) -> int {
            pf_norm_split_kernel<<<rows, PF_EW_THREADS, 0, s>>>(h, d, d, lw.g1, c.rms_eps, hi, lo, rs);
            int rr = pf_gemm(m, lw.wqkv, 3 * d, d, rows, qkv, nullptr, rs);
            if (rr != KG_OK) return rr;
            pf_rope_append_kernel<WT><<<dim3(rows, H), 64, 0, s>>>(D, qkv, b0, (WT*)D.kcache + (size_t)li * lstride, (WT*)D.vcache + (size_t)li * lstride);
            return KG_OK;
        };
        for (int i = 0; i < L; ++i) {
            const LayerW& lw = m->layers_host[i];
            if ((r = qkv_and_append(lw, i)) != KG_OK) return r;
            AttArgs at;
            at.qkv = qkv; at.M = 0; at.pos0 = b0; at.kc = (WT*)D.kcache + (size_t)i * lstride; at.vc = (WT*)D.vcache + (size_t)i * lstride;
            at.out = attn; at.opk = nullptr;
            pf_attention_kernel<<<m->nctas, NTHREADS, SMEM_TOTAL, s>>>(D, at, rows);
            pf_split_kernel<<<dim3(rows, (d / 4 + PF_EW_THREADS - 1) / PF_EW_THREADS), PF_EW_THREADS, 0, s>>>(attn, d, d, hi, lo);
            if ((r = pf_gemm(m, lw.wo, d, d, rows, h2, h, nullptr)) != KG_OK) return r;
            pf_norm_split_kernel<<<rows, PF_EW_THREADS, 0, s>>>(h2, d, d, lw.g2, c.rms_eps, hi, lo, rs);
            if ((r = pf_gemm(m, lw.wgate, F, d, rows, gate, nullptr, rs, lw.wup, up)) != KG_OK) return r;
            pf_swiglu_split_kernel<<<dim3(rows, (F / 4 + PF_EW_THREADS - 1) / PF_EW_THREADS), PF_EW_THREADS, 0, s>>>(gate, up, F, hi, lo);
            if ((r = pf_gemm(m, lw.wdown, d, F, rows, h, h2, nullptr)) != KG_OK) return r;
            if (i == c.exit_layer - 1 && (r = qkv_and_append(m->layers_host[L], L)) != KG_OK) return r;      // the adapter's K / V
        }
        CK(cudaGetLastError());
    }
    // LM head on the last prompt row (still in h): the decode path's fused head operator on one row
    {
        const int last = (n - 1) % PF_ROWS;
        pack_rows_kernel<<<m->nctas, 256, 0, s>>>(h + (size_t)last * d, d, 1, d, D.g_final, D.hA_pk, d * 4, D.ssq_hA, m->nctas);
        LinArgs a{};
        a.W = D.head; a.N = c.vocab; a.K = d; a.M = 1; a.x = h + (size_t)last * d; a.ldx = d; a.gain = D.g_final; a.eps = c.rms_eps;
        a.xpk = D.hA_pk; a.ldpk = d * 4; a.ssq_in = D.ssq_hA;
        a.epi = EPI_HEAD; a.scale = c.logit_scale; a.head_part = D.head_part;
        a.logits_dbg = c.debug_logits ? D.dbg_verify : nullptr; a.ld_dbg = c.vocab;
        op_linear_kernel<WT><<<m->nctas, BLOCK_THREADS, SMEM_TOTAL, s>>>(a, 1);
        pf_finish_kernel<<<1, 32, 0, s>>>(D.head_part, m->nctas, D.st, D.out_tokens, n, (const int*)(A + m->lay.off_pf_err));
        CK(cudaGetLastError());
    }
    return KG_OK;
}

}  // namespace

extern "C" int kg_debug_set_prefill_mode(kg_model* m, int mode) {
    if (!m || (mode != 0 && mode != 1)) return KG_E_ARG;
    m->prefill_mode = mode;
    return KG_OK;
}

extern "C" int kg_op_gemm(const void* W, int32_t N, int32_t K, const float* x, int32_t M, const float* resid, float* out,
                          void* scratch, void* stream) {
    if (!W || !x || !out || !scratch || M < 1 || N < 1 || K < 1) return KG_E_ARG;
    if (!aligned16(W) || !aligned16(x) || !aligned16(resid) || !aligned16(out) || !aligned16(scratch)) return KG_E_ARG;
    if (N % GM_BN || K % GM_BK) return KG_E_ARG;
    const int rows_pad = (M + GM_BM - 1) / GM_BM * GM_BM;
    OpScratch sc = op_layout();
    if ((size_t)rows_pad * K * 4 > 4 * (size_t)KG_M_MAX * S_CAP * 8192) return KG_E_LIMIT;  // both planes live in the split-partial scratch
    if (!encode_tiled_fn()) { std::snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled is not available"); return KG_E_CUDA; }
    cudaStream_t s = (cudaStream_t)stream;
    __nv_bfloat16* hi = (__nv_bfloat16*)((char*)scratch + sc.off_po);
    __nv_bfloat16* lo = hi + (size_t)rows_pad * K;
    int* err = (int*)((char*)scratch + sc.off_cnt);
    CK(cudaMemsetAsync(err, 0, 4, s));
    CK(cudaMemsetAsync(hi, 0, (size_t)rows_pad * K * 4, s));
    CK(cudaFuncSetAttribute((const void*)pf_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GM_SMEM));
    pf_split_kernel<<<dim3(M, (K / 4 + PF_EW_THREADS - 1) / PF_EW_THREADS), PF_EW_THREADS, 0, s>>>(x, K, K, hi, lo);
    CUtensorMap th, tl, tw;
    if (!make_tmap(&th, hi, rows_pad, K) || !make_tmap(&tl, lo, rows_pad, K) || !make_tmap(&tw, W, N, K)) {
        std::snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed");
        return KG_E_CUDA;
    }
    GemmArgs g;
    g.C = out; g.C2 = nullptr; g.ldc = N; g.resid = resid; g.ldr = N; g.rowscale = nullptr; g.rows = M; g.N = N; g.K = K; g.err = err;
    pf_gemm_kernel<<<dim3(N / GM_BN, rows_pad / GM_BM), GM_THREADS, GM_SMEM, s>>>(th, tl, tw, tw, g);
    CK(cudaGetLastError());
    return KG_OK;
}
