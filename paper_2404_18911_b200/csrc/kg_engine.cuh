// The persistent decode kernel: one cooperative grid (one CTA per SM) runs whole phases of the
// method - prefill chunks, the draft loop with its on-device exit test, the verify pass, the
// prefix accept / rollback, or many rounds back to back - with grid barriers between dependent
// operators and no host involvement.
//
// Every thread of every CTA walks the same operator sequence and holds the same copy of the
// sequence state.  The consumer warps do the arithmetic and take part in the grid barriers; the
// producer warp only issues the weight copies of each linear operator, so it runs ahead of the
// consumers (through barriers and attention) until the next decision that depends on a result
// (a drafted token, its confidence, the accepted prefix), which it receives through shared memory.
#pragma once

#include "kg_device.cuh"

namespace kg {

enum { PROG_PREFILL = 0, PROG_DRAFT = 1, PROG_VERIFY = 2, PROG_DECODE = 3, PROG_AR = 4 };

struct Program {
    int kind;
    int n;              // PREFILL: prompt length; DECODE / AR: total tokens wanted (x_0 included)
    float eta; int gamma; int stop_mode;
    int force_simple;   // 1: route bf16 linears through the plain path (cross-check)
    unsigned long long wait_clk;   // clocks after which a device-side wait gives up (KG_E_TIMEOUT)
    int skip_arrival;   // test hook: 1 + index of a CTA that leaves out its first grid-barrier arrival, so that a wait expires
};

#define KG_SYNC(where) do { if (!sync(where)) return false; } while (0)
#define KG_LIN(args) do { if (!linear(args)) return false; } while (0)

// Rows handed from one operator to the next: fp32 rows (residual input, plain path), their packed copy
// scaled by the reader's norm gain, and the per-CTA sums of squares the reader's RMSNorm needs.
struct ActIn { const float* x; const unsigned char* pk; const float* ssq; };
struct ActOut { float* x; PkOut pk[2]; float* ssq; };

// PROD: the instruction stream of the producer warp (it only issues weight copies and follows the control flow) or of
// the consumer warps; the two are compiled apart because they run with different register budgets.
template <typename WT, bool PROD>
struct Engine {
    const Dev& D;
    Ctx& c;
    const Program& pg;

    __device__ Engine(const Dev& d, Ctx& cx, const Program& p) : D(d), c(cx), pg(p) {}

    // ---- leaf operations: what a thread does depends on its role -------------------------------
    __device__ __forceinline__ bool streamed() const { return D.dm.stream != 0 && pg.force_simple == 0; }
    __device__ __forceinline__ bool sync(int where) { if constexpr (PROD) return true; else return grid_sync(c, where); }
    // this role's operator table in shared memory, and the one thread of the role that fills it
    __device__ __forceinline__ OpTable* table() const {
        if constexpr (PROD) __syncwarp();    // the lanes have left the previous operator before lane 0 rewrites the table
        return reinterpret_cast<OpTable*>(PROD ? c.ctl->tab_prod : c.ctl->tab_cons);
    }
    __device__ __forceinline__ bool writer() const { return PROD ? (threadIdx.x & 31) == 0 : threadIdx.x == 0; }
    __device__ __forceinline__ bool linear(const LinArgs* a, bool publish) {
        if constexpr (PROD) return linear_producer(a, c, streamed(), publish);
        else return linear_consumer<WT>(a, c, streamed(), publish);
    }
    __device__ __forceinline__ void attention(const AttArgs* at) { if constexpr (!PROD) attention_op<WT>(D, at, c); }

    __device__ size_t cache_layer_stride() const {
        return (size_t)D.dm.n_pages * D.dm.H * D.dm.page_size * D.dm.hd;
    }
    __device__ __forceinline__ size_t ldpk() const { return (size_t)D.dm.d * 4; }
    __device__ __forceinline__ ActIn act_h() const { return ActIn{D.h, D.hA_pk, D.ssq_hA}; }
    // the residual stream as an output, packed for a reader whose norm gain is `gain`
    __device__ __forceinline__ ActOut out_h(const float* gain) const {
        ActOut o; o.x = D.h; o.pk[0] = PkOut{gain, D.hA_pk}; o.pk[1] = PkOut{nullptr, nullptr}; o.ssq = D.ssq_hA; return o;
    }
    // norm gain of whatever reads the output of layer i: the next layer, or the LM head after the last one
    __device__ __forceinline__ const float* next_gain(int i) const { return i + 1 < D.dm.L ? D.layers[i + 1].g1 : D.g_final; }

    // an id outside [0, V) never indexes the embedding table (ids that arrive in device memory are checked by a
    // kernel of their own, which records the error; here the access is merely kept in bounds)
    __device__ __forceinline__ int safe_token(int tok) const { return (unsigned)tok < (unsigned)D.dm.V ? tok : 0; }

    // h[i] = E[token_i]; packed for layer 0
    __device__ void embed_rows(const int* toks_global, int tok_single, int M) {
        if constexpr (PROD) return;
        const int d = D.dm.d;
        const WT* E = reinterpret_cast<const WT*>(D.embed);
        if (!streamed()) {
            for (int idx = c.cta * NTHREADS + threadIdx.x; idx < M * d; idx += c.nctas * NTHREADS) {
                const int i = idx / d, e = idx % d;
                const int tok = safe_token(toks_global ? __ldcg(toks_global + i) : tok_single);
                D.h[idx] = wt_to_float<WT>(E[(size_t)tok * d + e]);
            }
            return;
        }
        LinArgs a{};
        a.N = d; a.M = M; a.out = D.h; a.ldo = d;
        a.pk[0] = PkOut{D.layers[0].g1, D.hA_pk}; a.ldpk_out = (int)ldpk(); a.ssq_out = D.ssq_hA;
        emit_plain_rows(a, c, [&](int m, int e) {
            const int tok = safe_token(toks_global ? __ldcg(toks_global + m) : tok_single);
            return wt_to_float<WT>(E[(size_t)tok * d + e]);
        });
    }

    // Arguments of the attention block of layer / adapter `li` on M rows at pos0: [0] q, k, v and [1] the output
    // projection with its residual, plus the attention itself.
    __device__ __forceinline__ void fill_attention_block(OpTable* t, const LayerW& lw, int li, int M, int pos0, const ActIn& in,
                                                         float* o_out, const PkOut& o_pk, float* o_ssq) {
        const Dims& dm = D.dm;
        LinArgs& q = t->lin[0];
        q = LinArgs{};
        q.M = M; q.eps = dm.eps;
        q.W = lw.wqkv; q.N = 3 * dm.d; q.K = dm.d;
        q.x = in.x; q.ldx = dm.d; q.gain = lw.g1; q.xpk = in.pk; q.ldpk = (int)ldpk(); q.ssq_in = in.ssq;
        q.epi = EPI_STORE; q.out = D.qkv; q.ldo = 3 * dm.d;
        AttArgs& at = t->att;
        at.qkv = D.qkv; at.M = M; at.pos0 = pos0;
        at.kc = reinterpret_cast<WT*>(D.kcache) + (size_t)li * cache_layer_stride();
        at.vc = reinterpret_cast<WT*>(D.vcache) + (size_t)li * cache_layer_stride();
        at.out = D.attn; at.opk = streamed() ? D.attn_pk : nullptr;
        LinArgs& o = t->lin[1];
        o = LinArgs{};
        o.M = M; o.eps = dm.eps;
        o.W = lw.wo; o.N = dm.d; o.K = dm.d; o.x = D.attn; o.ldx = dm.d;
        o.xpk = D.attn_pk; o.ldpk = (int)ldpk();
        o.epi = EPI_RESID; o.resid = in.x; o.ldr = dm.d; o.out = o_out; o.ldo = dm.d;
        o.pk[0] = o_pk; o.ldpk_out = (int)ldpk(); o.ssq_out = o_ssq;
    }

    // One decoder block on M rows at positions pos0.. (Section 3.1's M^b layers):
    //   h  = x + Wo Attn(RMSNorm(x; g1));   out = h + Wdown(SiLU(Wgate n) * Wup n), n = RMSNorm(h; g2)
    __device__ bool run_layer(int li, int M, int pos0, const ActIn& in, const ActOut& out) {
        const Dims& dm = D.dm;
        OpTable* t = table();
        if (writer()) {
            const LayerW lw = D.layers[li];
            fill_attention_block(t, lw, li, M, pos0, in, D.h, PkOut{lw.g2, D.hB_pk}, D.ssq_hB);
            LinArgs& gu = t->lin[2];
            gu = LinArgs{};
            gu.M = M; gu.eps = dm.eps;
            gu.W = lw.wgate; gu.W2 = lw.wup; gu.N = dm.F; gu.K = dm.d; gu.x = D.h; gu.ldx = dm.d; gu.gain = lw.g2;
            gu.xpk = D.hB_pk; gu.ldpk = (int)ldpk(); gu.ssq_in = D.ssq_hB;
            gu.epi = EPI_SWIGLU; gu.out = D.act; gu.ldo = dm.F;
            gu.pk[0] = PkOut{nullptr, D.act_pk}; gu.ldpk_out = dm.F * 4;
            LinArgs& dn = t->lin[3];
            dn = LinArgs{};
            dn.M = M; dn.eps = dm.eps;
            dn.W = lw.wdown; dn.N = dm.d; dn.K = dm.F; dn.x = D.act; dn.ldx = dm.F;
            dn.xpk = D.act_pk; dn.ldpk = dm.F * 4;
            dn.epi = EPI_RESID; dn.resid = D.h; dn.ldr = dm.d; dn.out = out.x; dn.ldo = dm.d;
            dn.pk[0] = out.pk[0]; dn.pk[1] = out.pk[1]; dn.ldpk_out = (int)ldpk(); dn.ssq_out = out.ssq;
        }
        if (!linear(&t->lin[0], true)) return false;
        KG_SYNC(10);
        attention(&t->att);
        KG_SYNC(11);
        if (!linear(&t->lin[1], false)) return false;
        KG_SYNC(12);
        if (!linear(&t->lin[2], false)) return false;
        KG_SYNC(13);
        if (!linear(&t->lin[3], false)) return false;
        KG_SYNC(14);
        return true;
    }

    // Adapter A (Section 3.1, Table 2): a = f + W^A_o Attn(RMSNorm(f; g_in)) on the rows `in` at pos0..;
    // with want_out == false only the adapter's K/V are appended (prefill).
    __device__ bool run_adapter(int M, int pos0, const ActIn& in, bool want_out) {
        const Dims& dm = D.dm;
        OpTable* t = table();
        if (writer()) {
            const LayerW lw = D.layers[dm.L];
            fill_attention_block(t, lw, dm.L, M, pos0, in, D.abuf, PkOut{lw.g2, D.abuf_pk}, D.ssq_abuf);
        }
        if (!linear(&t->lin[0], true)) return false;
        KG_SYNC(20);
        attention(&t->att);
        KG_SYNC(21);
        if (!want_out) return true;
        if (!linear(&t->lin[1], false)) return false;
        KG_SYNC(22);
        return true;
    }

    // Shared LM head on the rows `in` (norm gain `gain`), then the merged (token, p) per row: the same
    // values in every thread of every CTA, the producer warp included (it receives them through
    // shared memory and an mbarrier, which also holds it back until the result exists).
    __device__ bool run_head(const ActIn& in, int M, const float* gain, float* dbg, int* toks, float* ps) {
        const Dims& dm = D.dm;
        OpTable* t = table();
        if (writer()) {
            LinArgs& a = t->lin[0];
            a = LinArgs{};
            a.M = M; a.eps = dm.eps;
            a.W = D.head; a.N = dm.V; a.K = dm.d; a.x = in.x; a.ldx = dm.d; a.gain = gain;
            a.xpk = in.pk; a.ldpk = (int)ldpk(); a.ssq_in = in.ssq;
            a.epi = EPI_HEAD; a.scale = dm.logit_scale; a.head_part = D.head_part;
            a.logits_dbg = dm.debug ? dbg : nullptr; a.ld_dbg = dm.V;
        }
        if (!linear(&t->lin[0], true)) return false;
        if constexpr (PROD) {
            // held back here until the consumers have the result
            int ok = 1;
            const unsigned mp = c.mail_phase;
            if ((threadIdx.x & 31) == 0) ok = mbar_wait(c, &c.ctl->mail, mp, 42) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if ((threadIdx.x & 31) == 0) c.mail_phase = mp ^ 1u;      // the context is shared by the warp: one lane updates it
            __syncwarp();
            if (!ok) return false;
        } else {
            if (!grid_sync(c, 30)) return false;
            for (int m = threadIdx.x >> 5; m < M; m += NWARPS) {           // one warp per row
                int tk; float p;
                head_final_warp(D.head_part, c.nctas, m, tk, p);
                if ((threadIdx.x & 31) == 0) { c.ctl->head_tok[m] = tk; c.ctl->head_p[m] = p; }
            }
            cta_sync();
            if (threadIdx.x == 0) mbar_arrive(&c.ctl->mail);
        }
        for (int i = 0; i < M; ++i) { toks[i] = c.ctl->head_tok[i]; ps[i] = c.ctl->head_p[i]; }
        return true;
    }

    // ---- sequence state, replicated: every thread of every CTA holds the same values -----------
    int P, len_A, x0, total, rounds;
    int n_d, n_steps;
    int dtok[M_MAX];
    float dconf[M_MAX];

    __device__ void load_state() {
        P = __ldcg(&D.st->P); len_A = __ldcg(&D.st->len_A); x0 = __ldcg(&D.st->x0);
        total = __ldcg(&D.st->total); rounds = __ldcg(&D.st->rounds);
        n_d = __ldcg(&D.st->n_d); n_steps = __ldcg(&D.st->n_steps);
        for (int i = 0; i < M_MAX; ++i) { dtok[i] = __ldcg(&D.st->draft_tok[i]); dconf[i] = __ldcg(&D.st->conf[i]); }
    }
    __device__ bool leader() const { return c.cta == 0 && threadIdx.x == 0; }

    // the early-feature slot `slot` as an input of the adapter / of the first deep layer
    __device__ __forceinline__ ActIn feat_for_adapter(int slot) const {
        return ActIn{D.feat + (size_t)slot * D.dm.d, D.featA_pk + (size_t)slot * ldpk(), D.ssq_feat + (size_t)slot * c.nctas};
    }
    __device__ __forceinline__ ActIn feat_for_deep(int slot) const {
        return ActIn{D.feat + (size_t)slot * D.dm.d, D.featD_pk + (size_t)slot * ldpk(), D.ssq_feat + (size_t)slot * c.nctas};
    }

    // early feature of token `tok` at position pos -> feat slot (fp32 and packed for both of its readers)
    __device__ bool shallow_pass(int tok, int pos, int slot) {
        const Dims& dm = D.dm;
        embed_rows(nullptr, tok, 1);
        KG_SYNC(1);
        for (int i = 0; i < dm.l; ++i) {
            ActOut o = out_h(next_gain(i));
            if (i == dm.l - 1) {
                o.x = D.feat + (size_t)slot * dm.d;
                o.pk[0] = PkOut{D.layers[dm.L].g1, D.featA_pk + (size_t)slot * ldpk()};
                o.pk[1] = PkOut{D.layers[dm.l].g1, D.featD_pk + (size_t)slot * ldpk()};
                o.ssq = D.ssq_feat + (size_t)slot * c.nctas;
            }
            if (!run_layer(i, 1, pos, act_h(), o)) return false;
        }
        return true;
    }

    // Draft phase of one round (Section 3.2; Eq. 4; Figure 2).
    __device__ bool draft_phase() {
        const Dims& dm = D.dm;
        n_d = 0; n_steps = 0;
        int cur = x0;
        bool stop_after_shallow = false;
        while (true) {
            if (!shallow_pass(cur, P + n_d, 1 + n_d)) return false;                 // f[n_d]
            if (n_d == pg.gamma || stop_after_shallow) break;
            const int MA = P + n_d - len_A + 1;                                     // 1, or 2 when the adapter cache lags
            if (!run_adapter(MA, len_A, feat_for_adapter(1 + n_d - (MA - 1)), true)) return false;
            int tk[M_MAX]; float pp[M_MAX];
            const ActIn hin{D.abuf + (size_t)(MA - 1) * dm.d, D.abuf_pk + (size_t)(MA - 1) * ldpk(), D.ssq_abuf + (size_t)(MA - 1) * c.nctas};
            if (!run_head(hin, 1, D.layers[dm.L].g2, D.dbg_draft + (size_t)n_steps * dm.V, tk, pp)) return false;
            len_A += MA;
            dconf[n_steps] = pp[0];
            n_steps++;
            if (pg.stop_mode == 1 && pp[0] <= pg.eta) break;                        // drop the low-confidence token
            dtok[n_d] = tk[0];
            n_d++;
            cur = tk[0];
            if (pg.stop_mode == 0 && pp[0] <= pg.eta) stop_after_shallow = true;    // keep it; its feature is still needed
        }
        if (leader()) {
            State* st = D.st;
            st->n_d = n_d; st->n_steps = n_steps; st->len_A = len_A; st->pending = 1;
            for (int i = 0; i < M_MAX; ++i) { st->draft_tok[i] = dtok[i]; st->conf[i] = dconf[i]; }
            st->draft_steps_total += n_steps; st->drafted_total += n_d;
        }
        return true;
    }

    // Verify pass + prefix accept + rollback (Section 3: discard after the first reject; Figure 2).
    __device__ bool verify_phase() {
        const Dims& dm = D.dm;
        const int M = n_d + 1;
        for (int i = dm.l; i < dm.L; ++i)
            if (!run_layer(i, M, P, (i == dm.l) ? feat_for_deep(1) : act_h(), out_h(next_gain(i)))) return false;
        int t[M_MAX]; float pp[M_MAX];
        if (!run_head(act_h(), M, D.g_final, D.dbg_verify, t, pp)) return false;
        int k = 0;
        while (k < n_d && dtok[k] == t[k]) ++k;
        const int newP = P + k + 1;
        if (len_A > newP) len_A = newP;
        if (len_A < newP && !PROD) {
            // the adapter has not seen f[k] (k == n_d): keep it as the feature of position newP-1 (slot 0)
            const int gtid = c.cta * NTHREADS + threadIdx.x, gn = c.nctas * NTHREADS;
            const float* src = D.feat + (size_t)(1 + k) * dm.d;
            for (int e = gtid; e < dm.d; e += gn) D.feat[e] = __ldcg(src + e);
            const unsigned* psrc = reinterpret_cast<const unsigned*>(D.featA_pk + (size_t)(1 + k) * ldpk());
            unsigned* pdst = reinterpret_cast<unsigned*>(D.featA_pk);
            for (int e = gtid; e < dm.d; e += gn) pdst[e] = __ldcg(psrc + e);
            for (int e = gtid; e < c.nctas; e += gn) D.ssq_feat[e] = __ldcg(D.ssq_feat + (size_t)(1 + k) * c.nctas + e);
        }
        if (leader()) {
            State* st = D.st;
            for (int i = 0; i < k; ++i) { D.out_tokens[total + i] = dtok[i]; st->emitted[i] = dtok[i]; }
            D.out_tokens[total + k] = t[k]; st->emitted[k] = t[k];
            for (int i = 0; i < M; ++i) st->target[i] = t[i];
            D.S[rounds] = k + 1;
            D.round_log[rounds * 4 + 0] = n_d; D.round_log[rounds * 4 + 1] = n_steps;
            D.round_log[rounds * 4 + 2] = k; D.round_log[rounds * 4 + 3] = P;
            st->M = M; st->k_acc = k; st->n_emit = k + 1;
            st->P = newP; st->len_A = len_A; st->x0 = t[k]; st->pending = 0;
            st->total = total + k + 1; st->rounds = rounds + 1; st->accepted_total += k;
        }
        P = newP; x0 = t[k]; total += k + 1; rounds += 1;
        return true;
    }

    __device__ bool prefill() {
        const Dims& dm = D.dm;
        const int n = pg.n;
        int tk[M_MAX]; float pp[M_MAX];
        tk[0] = 0;
        for (int c0 = 0; c0 < n; c0 += M_MAX) {
            const int M = min(M_MAX, n - c0);
            embed_rows(D.prompt + c0, 0, M);
            KG_SYNC(2);
            for (int i = 0; i < dm.l; ++i) {
                ActOut o = out_h(next_gain(i));
                if (i == dm.l - 1) o.pk[1] = PkOut{D.layers[dm.L].g1, D.featA_pk};    // the adapter reads the same rows
                if (!run_layer(i, M, c0, act_h(), o)) return false;
            }
            if (!run_adapter(M, c0, ActIn{D.h, D.featA_pk, D.ssq_hA}, false)) return false;
            for (int i = dm.l; i < dm.L; ++i) if (!run_layer(i, M, c0, act_h(), out_h(next_gain(i)))) return false;
            if (c0 + M == n) {
                const ActIn hin{D.h + (size_t)(M - 1) * dm.d, D.hA_pk + (size_t)(M - 1) * ldpk(), D.ssq_hA + (size_t)(M - 1) * c.nctas};
                if (!run_head(hin, 1, D.g_final, D.dbg_verify, tk, pp)) return false;
            }
        }
        if (leader()) {
            State* st = D.st;
            st->P = n; st->len_A = n; st->x0 = tk[0]; st->pending = 0; st->total = 1; st->rounds = 0;
            D.out_tokens[0] = tk[0];
        }
        return true;
    }

    __device__ bool ar_decode() {
        const Dims& dm = D.dm;
        int tk[M_MAX]; float pp[M_MAX];
        while (total < pg.n) {
            embed_rows(nullptr, x0, 1);
            KG_SYNC(3);
            for (int i = 0; i < dm.L; ++i) if (!run_layer(i, 1, P, act_h(), out_h(next_gain(i)))) return false;
            if (!run_head(act_h(), 1, D.g_final, D.dbg_verify, tk, pp)) return false;
            if (leader()) {
                D.out_tokens[total] = tk[0];
                D.st->P = P + 1; D.st->x0 = tk[0]; D.st->total = total + 1; D.st->len_A = -1;
            }
            P += 1; x0 = tk[0]; total += 1;
        }
        return true;
    }

    __device__ bool run_program() {
        switch (pg.kind) {
            case PROG_PREFILL: return prefill();
            case PROG_DRAFT: return draft_phase();
            case PROG_VERIFY: return verify_phase();
            case PROG_AR: return ar_decode();
            case PROG_DECODE:
                while (total < pg.n) {
                    if (!draft_phase()) return false;
                    if (!verify_phase()) return false;
                }
                return true;
        }
        return true;
    }

    __device__ void run() {
        // the plain path streams nothing: its producer warp has no part in the launch
        if (PROD && !streamed()) return;
        load_state();
        const bool ok = run_program();
        if (!ok && PROD) ring_drain(c);
    }
};

template <typename WT>
__global__ void __launch_bounds__(DECODE_THREADS, 1) kg_persistent_kernel(const __grid_constant__ Dev D, const Program pg) {
    extern __shared__ __align__(128) char smem[];
    Ctx& c = ctx_init(smem, D.st, D.bar, true, pg.wait_clk, pg.skip_arrival);
    if (threadIdx.x >= NTHREADS) {
        // the producer's warpgroup: keeps what the copy loop needs and returns the rest of its registers
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(PRODUCER_REGS));
        if (threadIdx.x < BLOCK_THREADS) {
            Engine<WT, true> eng(D, c, pg);
            eng.run();
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(CONSUMER_REGS));
        Engine<WT, false> eng(D, c, pg);
        eng.run();
    }
}

}  // namespace kg
