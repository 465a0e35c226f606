/* kangaroo.h - C ABI of the B200 (sm_100a) implementation of the Kangaroo batch-1
 * self-speculative decode step (Liu et al., "Kangaroo: Lossless Self-Speculative Decoding
 * via Double Early Exiting").
 *
 * The library owns no memory: the caller hands in one device arena and one CUDA stream, and
 * every kernel runs on that stream.  No call allocates device memory or creates streams.
 * All functions return KG_OK (0) or a negative kg_status; none throws or aborts.  Argument and
 * state errors launch nothing.
 *
 * Pointer suffixes: _host = host memory, _dev = device memory on the current device.
 *
 * Model (Section 3.1, Figure 2 of the paper): target M^b = LLaMA-style decoder with L layers;
 * self-draft model M^s = A o M^b[:l] (first l layers + adapter A = one attention with an input
 * and a last RMS norm) re-using the target's LM head.  Matrices are row-major
 * [out_features, in_features]; W_qkv is [3d, d] (q rows, then k rows, then v rows).
 */
#ifndef KANGAROO_H_
#define KANGAROO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KG_M_MAX 16               /* most rows one pass may carry: gamma_max + 1 <= KG_M_MAX */
#define KG_GAMMA_MAX (KG_M_MAX - 1)

typedef enum {
    KG_OK = 0,
    KG_E_ARG = -1,       /* NULL pointer, bad size, unsupported shape */
    KG_E_STATE = -2,     /* call order violated (e.g. kg_verify without a pending draft) */
    KG_E_NOMEM = -3,     /* arena too small */
    KG_E_SEQ_FULL = -4,  /* the sequence would exceed max_seq */
    KG_E_CUDA = -5,      /* a CUDA runtime call failed */
    KG_E_TIMEOUT = -6,   /* a bounded device-side wait expired; the model must be re-initialised (kg_init_model) */
    KG_E_LIMIT = -7,     /* a size exceeds what a fixed-capacity entry point (kg_op_lm_head_noalloc) can hold */
    KG_E_INTERNAL = -8   /* a kernel found an index outside its table (e.g. a page number), skipped the access and
                            recorded it; kg_last_cuda_error() says which check; the model must be re-initialised */
} kg_status;

enum { KG_F32 = 0, KG_BF16 = 1 };            /* storage type of weights and KV cache */
enum { KG_STOP_KEEP = 0, KG_STOP_DROP = 1 }; /* is the draft whose confidence is <= eta kept? */

typedef struct kg_model kg_model;            /* opaque host handle */

typedef struct {
    uint32_t struct_size;                    /* = sizeof(kg_config) */
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;   /* L, d, H, hd, F, V */
    int32_t exit_layer;                      /* l, 1 <= l < L (Section 3.1) */
    int32_t dtype;                           /* KG_F32 | KG_BF16 */
    float rms_eps, rope_theta, logit_scale;  /* logits z = logit_scale * W_head y */
    int32_t max_seq, page_size, gamma_max;   /* KV capacity in tokens; tokens per KV page (a power of two); largest gamma */
    int32_t debug_logits;                    /* 1: keep every computed logit row in HBM for kg_debug_logits */
    int32_t page_shuffle;                    /* 1: non-identity page table (exercises the indirection) */
    /* synthetic initialisation, used when kg_init_model gets weights == NULL */
    uint64_t seed;
    float init_std, embed_std, deep_resid_scale, adapter_resid_scale, gain_std;
} kg_config;

/* Borrowed device pointers to caller-provided weights (optional), each 16-byte aligned (else KG_E_ARG:
 * the kernels read them with 16-byte bulk copies).  Arrays are HOST arrays of device pointers.  Index L (= n_layers) of wqkv / wo / g1 / g2 is the adapter (g1 = input norm
 * gain, g2 = last norm gain).  Matrices have the model's storage dtype, gains are fp32. */
typedef struct {
    const void* embed_dev;                   /* [V, d] */
    const void* head_dev;                    /* [V, d] */
    const float* g_final_dev;                /* [d] */
    const void* const* wqkv_dev;             /* L+1 x [3d, d] */
    const void* const* wo_dev;               /* L+1 x [d, d] */
    const void* const* wgate_dev;            /* L   x [F, d] */
    const void* const* wup_dev;              /* L   x [F, d] */
    const void* const* wdown_dev;            /* L   x [d, F] */
    const float* const* g1_dev;              /* L+1 x [d] */
    const float* const* g2_dev;              /* L+1 x [d] */
} kg_weights;

typedef struct {
    int32_t n_drafted;                       /* n_d: drafts kept this round */
    int32_t n_steps;                         /* adapter+head passes run (= confidences computed) */
    int32_t tokens[KG_GAMMA_MAX];            /* x'_1 .. x'_{n_d} */
    float conf[KG_GAMMA_MAX];                /* every confidence computed, a dropped token's included */
} kg_draft_out;

typedef struct {
    int32_t n_rows;                          /* M = n_d + 1 rows verified */
    int32_t n_accept;                        /* k: accepted drafts */
    int32_t n_emitted;                       /* k + 1 */
    int32_t emitted[KG_M_MAX];               /* x'_1..x'_k, t_k */
    int32_t target[KG_M_MAX];                /* t_0 .. t_{n_d}: the target's greedy token per row */
} kg_verify_out;

typedef struct {
    int32_t rounds;                          /* |S| */
    int32_t tokens;                          /* sum of S (tokens produced by rounds; x_0 of prefill not counted) */
    int32_t draft_steps;                     /* adapter+head passes in total */
    int32_t drafted;                         /* drafts kept in total */
    int32_t accepted;                        /* drafts accepted in total */
    double cr;                               /* Eq. 1 */
    double ctar[KG_M_MAX + 1];               /* Eq. 2 for w = 0 .. KG_M_MAX */
    float ms_decode;                         /* device time of the decode loop (CUDA events), 0 if not measured */
} kg_stats;

/* Bytes of arena kg_init_model needs: KV pages, activations, scratch, and (own_weights != 0)
 * the synthetic weights themselves.  Returns 0 on an invalid config. */
size_t kg_workspace_bytes(const kg_config* cfg, int own_weights);

/* Builds a model inside `arena_dev` (256-byte aligned, >= kg_workspace_bytes).  weights == NULL:
 * fills seeded synthetic weights on the device with the counter-based generator (bit-identical
 * to the host generator of the test inputs).  The arena and the stream stay owned by the caller
 * and must outlive the model.  `cuda_stream` is a cudaStream_t. */
int kg_init_model(const kg_config* cfg, const kg_weights* weights, void* arena_dev, size_t arena_bytes,
                  void* cuda_stream, kg_model** out);
int kg_free_model(kg_model* m);              /* frees the host handle only */

/* Forget the sequence (KV lengths, round state); weights stay. */
int kg_reset(kg_model* m);

/* All L layers over the prompt, the adapter's K/V for every prompt position, and
 * x_0 = argmax M^b(. | prompt) (Figure 2's starting point).  Requires a reset model.
 * kg_prefill copies the prompt from the host (ids outside [0, vocab) -> KG_E_ARG, nothing launched); if
 * first_token_host != NULL it synchronises the stream and returns x_0.  kg_prefill_device reads prompt ids
 * already in device memory and never synchronises: an id outside [0, vocab) is caught on the device (the
 * embedding lookup stays in bounds) and the next call that synchronises returns KG_E_ARG; kg_reset clears it. */
int kg_prefill(kg_model* m, const int32_t* prompt_host, int32_t n, int32_t* first_token_host);
int kg_prefill_device(kg_model* m, const int32_t* prompt_dev, int32_t n);

/* One round's draft phase (Section 3.2, Eq. 4; Figure 2): run M^s one token at a time from x_0,
 * stop when the top-1 probability p <= eta or gamma tokens are drafted; the early features
 * f_0..f_{n_d} stay on the device for kg_verify.  The whole loop, its exit test included, runs on
 * the device.  out (nullable): copies the result and synchronises the stream. */
int kg_draft(kg_model* m, float eta, int32_t gamma, int32_t stop_mode, kg_draft_out* out);

/* Verify the pending unit [f_0..f_{n_d}] with layers l+1..L in one pass, accept the longest
 * prefix of drafts that equals the target's greedy tokens, discard the rest, roll the KV caches
 * back (Section 3; Figure 2).  out (nullable): copies the result and synchronises. */
int kg_verify(kg_model* m, kg_verify_out* out);

/* Device-resident decode loop: rounds of draft + verify + accept until at least max_new tokens
 * (x_0 included) exist; one kernel launch, no host round-trip.  Requires a prefilled model.
 * stats (nullable): synchronises and fills it. */
int kg_decode(kg_model* m, int32_t max_new, float eta, int32_t gamma, int32_t stop_mode, kg_stats* stats);

/* Plain greedy autoregressive decoding of the target (the definition Kangaroo must reproduce,
 * Section 1): n_tokens tokens in total, x_0 included.  out_host (nullable) receives them. */
int kg_decode_ar(kg_model* m, int32_t n_tokens, int32_t* out_host);

/* reset + prefill + decode + read-back.  Returns exactly max_new tokens (x_0 first); the last
 * round is truncated so that sum(S) counts only returned tokens (Section 3, list S). */
int kg_generate(kg_model* m, const int32_t* prompt_host, int32_t n_prompt, int32_t max_new,
                float eta, int32_t gamma, int32_t stop_mode,
                int32_t* out_tokens_host, int32_t* n_out, kg_stats* stats);

/* Copies tokens produced so far (x_0 first) / the accepted-length list S to the host; synchronises. */
int kg_read_tokens(kg_model* m, int32_t* out_host, int32_t max_n, int32_t* n_out);
int kg_read_S(kg_model* m, int32_t* out_host, int32_t max_n, int32_t* n_out);

/* Per-round record of the rounds run so far, four int32 per round: n_d (drafts kept), n_steps
 * (adapter+head passes), k (drafts accepted), P (position of the round's x_0, Figure 2).  Copies at
 * most max_rounds records to out_host[max_rounds * 4]; synchronises. */
int kg_read_round_log(kg_model* m, int32_t* out_host, int32_t max_rounds, int32_t* n_out);

/* Parity helpers (need cfg.debug_logits = 1).  which = 0: draft logits of step `row` of the last
 * round; which = 1: verify / AR / prefill logits of row `row` of the last pass.  Copies V floats. */
int kg_debug_logits(kg_model* m, int32_t which, int32_t row, float* out_host);

/* Reads `count` elements starting at `offset` of a weight tensor, widened to fp32.
 * name: "embed","head","wqkv","wo","wgate","wup","wdown","g1","g2","g_final"; layer = L for the adapter. */
int kg_read_weight(kg_model* m, const char* name, int32_t layer, uint64_t offset, uint64_t count, float* out_host);

/* Microbenchmark support (the verify-step / draft-step shapes of the evaluation): pretend the
 * sequence has T tokens by filling every KV cache [0, T) with seeded N(0,1) entries, sets
 * x_0 = token, and, if n_d >= 0, a pending draft of n_d seeded tokens with N(0,1) early features. */
int kg_debug_fill_state(kg_model* m, int32_t T, int32_t n_d, uint64_t seed);

/* ---- test hooks (no part of the method; used by the parity and failure-path tests) ----------------
 * kg_debug_force_simple: route a bf16 model's linear operators through the plain (non tensor-core) path, a
 *   cross-check of the streamed path; KG_E_ARG for shapes whose 16 rows of max(d, F) floats do not fit in shared memory.  kg_debug_force_simple_ops: the same for the single-operator calls.
 * kg_debug_set_wait_budget: every wait inside a kernel (grid barrier, weight ring) gives up after this many
 *   milliseconds (default about 3 s) and the launch ends with KG_E_TIMEOUT in the state word.
 * kg_debug_skip_barrier_arrival: in the NEXT launch, CTA `cta` leaves out its first grid-barrier arrival, so that
 *   every CTA's wait runs into the budget: the host-injected way to exercise the time-out path.  Nothing traps or
 *   faults; all CTAs return, the stream stays usable, and the model answers KG_E_TIMEOUT until it is re-initialised. */
int kg_debug_force_simple(kg_model* m, int on);
int kg_debug_force_simple_ops(int on);
int kg_debug_set_wait_budget(kg_model* m, double milliseconds);
int kg_debug_skip_barrier_arrival(kg_model* m, int cta);
/* kg_debug_set_prefill_mode: 0 (default): prompts of 32 tokens and more take the tensor-core prompt pass when the
 *   model is bf16 with head_dim 64 / 128 and d, F multiples of 128; 1: every prompt takes the 16-row chunked pass of
 *   the decode kernels (the two are compared with each other and with the oracle in the tests). */
int kg_debug_set_prefill_mode(kg_model* m, int mode);

/* ---- single operators on caller buffers (unit tests and microbenchmarks) ------------------------
 * All pointers are device pointers, 16-byte aligned (int32 arrays: 4-byte), else KG_E_ARG; `scratch_dev` must hold
 * kg_op_scratch_bytes() bytes; the call is asynchronous on `cuda_stream`.  dtype is KG_F32 or KG_BF16 and is the type of W / KV. */
size_t kg_op_scratch_bytes(void);

/* out[M, N] = (resid ? resid : 0) + RMSNorm(x; gain, eps) W^T   (gain == NULL: no norm)
 * swiglu != 0: W is W_gate, W2 is W_up (both [N, K]) and out = SiLU(gate) * up. */
int kg_op_linear(int32_t dtype, const void* W_dev, const void* W2_dev, int32_t N, int32_t K,
                 const float* x_dev, int32_t M, const float* gain_dev, float eps,
                 const float* resid_dev, int32_t swiglu, float* out_dev,
                 void* scratch_dev, void* cuda_stream);

/* Fused LM head (Figure 2: shared head; Eq. 4's confidence): z = logit_scale * RMSNorm(x) W_head^T,
 * per row the arg max (lowest index on ties) and p = 1 / sum_i exp(z_i - z_max).
 * logits_dev (nullable) receives z [M, V]. */
int kg_op_lm_head(int32_t dtype, const void* W_head_dev, int32_t V, int32_t K, const float* x_dev, int32_t M,
                  const float* gain_dev, float eps, float logit_scale,
                  int32_t* tok_dev, float* p_dev, float* logits_dev, void* scratch_dev, void* cuda_stream);

/* kg_op_lm_head without any caller scratch and without any allocation (the paper has no counterpart: this is
 * a deployment convenience).  It is for callers that cannot obtain device memory at the time of the call -
 * code running while a memory pool is frozen or exhausted, inside a plugin whose host forbids cudaMalloc, or
 * in an error path that must still produce a token.  The per-CTA partial results that kg_op_lm_head keeps in
 * `scratch_dev` (per-CTA partial results, and the repacked copy of the input rows) live here in a 592 KB array
 * that is part of the library image, so every GPU that loads the library holds those 592 KB until the process exits.
 * Limits: M <= KG_M_MAX rows, K <= 8192 and a device with at most 256 SMs; anything larger returns KG_E_LIMIT.
 * V is not limited: W, x and the outputs remain caller memory.
 * The first call on each device looks up the array's device address (no allocation); make that first call
 * outside any stream capture.  All calls share the one array: two calls whose kernels overlap on the GPU
 * (different streams, no ordering between them) race on it and give wrong results; calls ordered on one
 * stream are safe, and nothing in the array has to be cleared between calls because every partial is
 * rewritten before it is read. */
int kg_op_lm_head_noalloc(int32_t dtype, const void* W_head_dev, int32_t V, int32_t K, const float* x_dev, int32_t M,
                          const float* gain_dev, float eps, float logit_scale,
                          int32_t* tok_dev, float* p_dev, float* logits_dev, void* cuda_stream);

/* The GEMM of the tensor-core prompt pass (the state Figure 2 starts from is built with it): out[M, N] = (resid ? resid : 0)
 * + x W^T for bf16 W [N, K] and fp32 x [M, K], any M >= 1; x is split into two bf16 planes (x = hi + lo) and both are
 * multiplied with W on the tensor cores into fp32.  N a multiple of 128, K a multiple of 64 (else KG_E_ARG);
 * ceil(M / 128) * 128 * K <= 2097152 elements so that the planes fit in `scratch_dev` (else KG_E_LIMIT). */
int kg_op_gemm(const void* W_dev, int32_t N, int32_t K, const float* x_dev, int32_t M, const float* resid_dev, float* out_dev,
               void* scratch_dev, void* cuda_stream);

/* Causal attention of M new rows at positions pos0.. over a paged KV cache (RoPE fused): takes the
 * raw q,k,v rows qkv[M, 3d], rotates q and k, appends k and v to the cache pages, and returns
 * out[M, d] = concat_heads softmax(q K^T / sqrt(hd)) V.  Cache layout: [page][head][slot][hd]. */
int kg_op_attention(int32_t dtype, const float* qkv_dev, int32_t M, int32_t pos0, int32_t n_heads, int32_t head_dim,
                    float rope_theta, void* kcache_dev, void* vcache_dev, const int32_t* page_table_dev,
                    int32_t page_size, float* out_dev, void* scratch_dev, void* cuda_stream);

const char* kg_strerror(int status);
/* After a call of this thread returned KG_E_CUDA: which CUDA runtime call failed and the runtime's name and text
 * for the error ("" if none failed yet).  The string is owned by the library and valid until the next failure. */
const char* kg_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* KANGAROO_H_ */
