// Online-softmax reducer over a stored relation (paper Section 5 "Online softmax"; attention
// appendix): the edge function supplies a score and a value,
//     s_e = scale * <q_d(e), k_s(e)>,   y_i = sum_e exp(s_e) v_s(e) / sum_e exp(s_e)  over row i,
// and the relation decides which interactions exist (a triangular relation is causal attention,
// an arbitrary CSR is graph attention).
//
// Same schedule as the sum / max reducers: merge-path tiles of "row ends + edges", one CTA per
// tile, edges split evenly over workers of G lanes, each lane owning 16 bytes of the query, key
// and value rows.  A worker walks its span in edge order with the streaming state of Section 5
// in registers: running maximum m (in units of log 2), mass l, accumulator o.  Four edges are
// taken per step: four key rows and four value rows are gathered at once, the four dot products
// are reduced over the worker's lanes by shuffles, the state is rescaled once per step.  Partial
// states at the ends of a span go to shared memory and are combined in edge order with the
// paper's rule  m = max(ma, mb), l = e^(ma-m) la + e^(mb-m) lb, o likewise;  a tile's trailing
// partial row is a carry-out in the workspace.  A finished row is stored finalised (o / l and
// lse = m + log l); since a finalised row is the state (lse, 1, y), the fix-up kernel can combine
// carry-outs of earlier tiles with it.  No atomics: results are reproducible.
#include "csr_shared.cuh"
#include <math.h>

namespace tiga {

constexpr float ATT_NEG_INF = -INFINITY;
constexpr float ATT_LOG2E = 1.4426950408889634f;
constexpr float ATT_LN2 = 0.6931471805599453f;

static __device__ __forceinline__ float att_exp2(float x) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

struct AttState {
    float m, l;
    float o[4];
    __device__ __forceinline__ void reset() { m = ATT_NEG_INF; l = 0.f; o[0] = o[1] = o[2] = o[3] = 0.f; }
    // fold a state that comes later in edge order (the paper's combine rule)
    __device__ __forceinline__ void combine(const float mb, const float lb, const float4 ob) {
        if (mb == ATT_NEG_INF) return;
        const float M = fmaxf(m, mb);
        const float ca = att_exp2(m - M), cb = att_exp2(mb - M);      // exp2(-inf) = 0 covers an empty left side
        l = fmaf(l, ca, lb * cb);
        o[0] = fmaf(o[0], ca, ob.x * cb); o[1] = fmaf(o[1], ca, ob.y * cb);
        o[2] = fmaf(o[2], ca, ob.z * cb); o[3] = fmaf(o[3], ca, ob.w * cb);
        m = M;
    }
};

// EXACT: the row fills the worker exactly (D == 4 G): constant row stride, no lane predicates.
template <int G, typename IT, bool EXACT>
__global__ void __launch_bounds__(CSR_THREADS) csr_attention_kernel(const CsrParams p) {
    constexpr int NW = CSR_THREADS / G;          // workers per CTA
    constexpr int LV = G * 4;                    // floats of one partial accumulator
    constexpr int U = 4;                         // edges per step

    __shared__ int s_ptr[CSR_TILE_ATT + 2];
    __shared__ __align__(16) int s_col[CSR_TILE_ATT + CSR_PAD];
    __shared__ __align__(16) float s_w[CSR_TILE_ATT + CSR_PAD];
    __shared__ long long s_coord[2];
    __shared__ int s_tag[2 * NW];                // local row of head (even) / tail (odd) partial, -1 = none
    __shared__ unsigned char s_first[NW];        // tail partial starts its chain
    __shared__ float s_pm[2 * NW], s_pl[2 * NW];
    extern __shared__ __align__(16) unsigned char s_dyn[];
    float* s_pv = reinterpret_cast<float*>(s_dyn);              // [2*NW][LV]

    const Tile t = stage_tile<IT, false, CSR_TILE_ATT>(p, s_ptr, s_col, s_w, s_coord);
    const int wk = threadIdx.x / G;
    const int ln = threadIdx.x % G;
    const unsigned wmask = G == 32 ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) / G * G));
    const unsigned nvec = EXACT ? (unsigned)G : (unsigned)p.nvec;
    const int F = EXACT ? 4 * G : p.F;
    const bool act = EXACT ? true : ln < p.nvec;
    const float4* __restrict__ qlane = reinterpret_cast<const float4*>(p.q) + ln;
    const float4* __restrict__ klane = reinterpret_cast<const float4*>(p.key) + ln;
    const float4* __restrict__ vlane = reinterpret_cast<const float4*>(p.x) + ln;
    const float sc2 = p.scale * ATT_LOG2E;       // scores in units of log 2
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

    auto load_q = [&](int r_local) { return act ? __ldg(qlane + (unsigned long long)(t.i0 + r_local) * nvec) : zero4; };
    auto dot_all = [&](float s) {                // sum over the worker's lanes, result in every lane
#pragma unroll
        for (int o = G / 2; o > 0; o >>= 1) s += __shfl_xor_sync(wmask, s, o);
        return s;
    };
    auto store_row = [&](long long row, const AttState& s) {
        const float inv = s.l > 0.f ? 1.f / s.l : 0.f;
        if (act) st_stream(reinterpret_cast<float4*>(p.out + row * F) + ln, make_float4(s.o[0] * inv, s.o[1] * inv, s.o[2] * inv, s.o[3] * inv));
        if (ln == 0) {
            const float lse = s.l > 0.f ? (s.m + log2f(s.l)) * ATT_LN2 : ATT_NEG_INF;
            p.gw[row] = lse;                     // workspace copy, read by the fix-up
            if (p.lse) p.lse[row] = lse;
        }
    };
    auto store_partial = [&](int entry, const AttState& s) {
#pragma unroll
        for (int k = 0; k < 4; ++k) s_pv[entry * LV + ln * 4 + k] = s.o[k];
        if (ln == 0) { s_pm[entry] = s.m; s_pl[entry] = s.l; }
    };
    auto merge_partial = [&](int entry, AttState& s) {
        s.combine(s_pm[entry], s_pl[entry], *reinterpret_cast<const float4*>(s_pv + entry * LV + ln * 4));
    };

    // rows that end in this tile without an edge in it: the empty state, finalised to the zero vector
    {
        AttState idn;
        idn.reset();
        for (int k = wk; k < t.nfin; k += NW) {
            const int ls = s_ptr[k] < 0 ? 0 : s_ptr[k];
            if (s_ptr[k + 1] == ls) store_row(t.i0 + k, idn);
        }
    }

    if (ln == 0) { s_tag[2 * wk] = -1; s_tag[2 * wk + 1] = -1; s_first[wk] = 0; }
    if (threadIdx.x == 0) p.carry_row[blockIdx.x] = -1;

    // spans start on multiples of U, so a step's U indices are one vector load
    const int chunk = ((t.ne + NW - 1) / NW + U - 1) / U * U;
    const int a = wk * chunk;
    const int b = (a + chunk < t.ne) ? a + chunk : t.ne;

    AttState st;
    st.reset();
    int r = 0;
    bool tail_valid = false, tail_first = false;
    if (a < b) {
        r = row_of_edge(s_ptr, t.nrows, a);
        int cur_end = s_ptr[r + 1];
        bool head = (s_ptr[r] < 0 ? 0 : s_ptr[r]) < a;   // the row began in an earlier span of this tile
        float4 qv = load_q(r);
        for (int e = a; e < b; e += U) {
            float4 kv[U], vv[U];
            // entries past the span are readable (next worker's edges or the pad) and never used
            const int4 c4 = *reinterpret_cast<const int4*>(s_col + e);
            const int cv[U] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned long long off = (unsigned long long)(unsigned)cv[u] * nvec;
                kv[u] = act ? __ldg(klane + off) : zero4;
                vv[u] = act ? __ldg(vlane + off) : zero4;
            }
            if (e + U <= b && e + U <= cur_end) {
                // common case: the whole step lies inside the current row and the span
                float s[U];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    s[u] = fmaf(qv.w, kv[u].w, fmaf(qv.z, kv[u].z, fmaf(qv.y, kv[u].y, qv.x * kv[u].x)));
#pragma unroll
                for (int o = G / 2; o > 0; o >>= 1)
#pragma unroll
                    for (int u = 0; u < U; ++u) s[u] += __shfl_xor_sync(wmask, s[u], o);
                float M = st.m;
#pragma unroll
                for (int u = 0; u < U; ++u) { s[u] *= sc2; M = fmaxf(M, s[u]); }
                const float c = att_exp2(st.m - M);
                st.l *= c; st.o[0] *= c; st.o[1] *= c; st.o[2] *= c; st.o[3] *= c;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float pr = att_exp2(s[u] - M);
                    st.l += pr;
                    st.o[0] = fmaf(pr, vv[u].x, st.o[0]); st.o[1] = fmaf(pr, vv[u].y, st.o[1]);
                    st.o[2] = fmaf(pr, vv[u].z, st.o[2]); st.o[3] = fmaf(pr, vv[u].w, st.o[3]);
                }
                st.m = M;
                continue;
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (e + u < b) {
                    if (e + u >= cur_end) {
                        // the current row is complete inside this span
                        if (head) { store_partial(2 * wk, st); if (ln == 0) s_tag[2 * wk] = r; }
                        else store_row(t.i0 + r, st);
                        st.reset();
                        head = false;
                        do { ++r; cur_end = s_ptr[r + 1]; } while (e + u >= cur_end);   // skip empty rows
                        qv = load_q(r);
                    }
                    const float s = sc2 * dot_all(fmaf(qv.w, kv[u].w, fmaf(qv.z, kv[u].z, fmaf(qv.y, kv[u].y, qv.x * kv[u].x))));
                    const float M = fmaxf(st.m, s);
                    const float c = att_exp2(st.m - M), pr = att_exp2(s - M);
                    st.l = fmaf(st.l, c, pr);
                    st.o[0] = fmaf(st.o[0], c, pr * vv[u].x); st.o[1] = fmaf(st.o[1], c, pr * vv[u].y);
                    st.o[2] = fmaf(st.o[2], c, pr * vv[u].z); st.o[3] = fmaf(st.o[3], c, pr * vv[u].w);
                    st.m = M;
                }
            }
        }
        if (cur_end <= b) {
            if (head) { store_partial(2 * wk, st); if (ln == 0) s_tag[2 * wk] = r; }
            else store_row(t.i0 + r, st);
        } else {
            // the row continues past this span: tail partial
            tail_valid = true;
            tail_first = !head;
            store_partial(2 * wk + 1, st);
            if (ln == 0) { s_tag[2 * wk + 1] = r; s_first[wk] = tail_first ? 1 : 0; }
        }
    }
    __syncthreads();

    // combine chains of partial states in edge order; the worker that opens a chain owns it
    if (tail_valid && tail_first) {
        bool finished = false;
        for (int w2 = wk + 1; w2 < NW; ++w2) {
            if (s_tag[2 * w2] == r) { merge_partial(2 * w2, st); finished = true; break; }
            if (s_tag[2 * w2 + 1] == r && !s_first[w2]) merge_partial(2 * w2 + 1, st);
            else break;
        }
        if (finished) {
            store_row(t.i0 + r, st);
        } else {
            // trailing unfinished row of the tile -> carry-out
            if (ln == 0) {
                p.carry_row[blockIdx.x] = (int32_t)(t.i0 + r);
                p.carry_ml[blockIdx.x] = make_float2(st.m, st.l);
            }
            if (act) *(reinterpret_cast<float4*>(p.carry_val + (size_t)blockIdx.x * F) + ln) = make_float4(st.o[0], st.o[1], st.o[2], st.o[3]);
        }
    }
}

// Combine the carry-outs of consecutive tiles that belong to one row, in edge order, with the part
// of the row stored by the tile it ends in (a finalised row is the state (lse, 1, y)), and finalise.
// One thread per (tile, feature); only the first tile of a run does the work.
__global__ void csr_attention_fixup_kernel(const CsrParams p) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long tile = idx / p.F;
    const int f = (int)(idx % p.F);
    if (tile >= p.ntiles) return;
    const int row = p.carry_row[tile];
    if (row < 0) return;
    if (tile > 0 && p.carry_row[tile - 1] == row) return;
    float m = p.carry_ml[tile].x, l = p.carry_ml[tile].y, o = p.carry_val[tile * p.F + f];
    auto combine = [&](const float mb, const float lb, const float ob) {
        if (mb == ATT_NEG_INF) return;
        const float M = fmaxf(m, mb);
        const float ca = att_exp2(m - M), cb = att_exp2(mb - M);
        l = fmaf(l, ca, lb * cb);
        o = fmaf(o, ca, ob * cb);
        m = M;
    };
    for (long long u = tile + 1; u < p.ntiles && p.carry_row[u] == row; ++u)
        combine(p.carry_ml[u].x, p.carry_ml[u].y, p.carry_val[u * p.F + f]);
    const float lse_tail = p.gw[row];
    combine(lse_tail * ATT_LOG2E, 1.f, p.out[(size_t)row * p.F + f]);
    p.out[(size_t)row * p.F + f] = o / l;
    if (f == 0 && p.lse) p.lse[row] = (m + log2f(l)) * ATT_LN2;
}

template <int G, typename IT>
static tiga_status launch_attention_t(const CsrParams& p, cudaStream_t s) {
    constexpr int smem = 2 * (CSR_THREADS / G) * G * 4 * (int)sizeof(float);
    if (p.nvec == G) csr_attention_kernel<G, IT, true><<<counted((unsigned)p.ntiles), CSR_THREADS, smem, s>>>(p);
    else csr_attention_kernel<G, IT, false><<<counted((unsigned)p.ntiles), CSR_THREADS, smem, s>>>(p);
    const long long work = p.ntiles * p.F;
    csr_attention_fixup_kernel<<<counted((unsigned)((work + 255) / 256)), 256, 0, s>>>(p);
    return launch_status();
}

template <typename IT>
static tiga_status launch_attention(const CsrParams& p, cudaStream_t s) {
    if (p.nvec <= 4) return launch_attention_t<4, IT>(p, s);
    if (p.nvec <= 8) return launch_attention_t<8, IT>(p, s);
    if (p.nvec <= 16) return launch_attention_t<16, IT>(p, s);
    return launch_attention_t<32, IT>(p, s);
}

static tiga_status attention_check(const tiga_csr* g, int32_t D) {
    if (!g || g->n_dst < 0 || g->n_src < 0 || g->n_edges < 0) return TIGA_ERR_INVALID_ARG;
    if (g->rowptr_type != TIGA_I32 && g->rowptr_type != TIGA_I64) return TIGA_ERR_INVALID_ARG;
    if (g->rowptr_type == TIGA_I32 && g->n_edges > 0x7fffffffLL) return TIGA_ERR_INVALID_ARG;
    if (D < 4 || (D & 3)) return TIGA_ERR_INVALID_ARG;
    if (D > 128) return TIGA_ERR_UNSUPPORTED;
    if (g->n_dst > 0x7fffffffLL || g->n_src > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    if ((g->n_dst + g->n_edges + CSR_TILE_ATT - 1) / CSR_TILE_ATT > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    return TIGA_OK;
}

static size_t attention_carve(CsrParams* p, void* ws) {
    Carver cv(ws);
    p->carry_row = cv.take<int32_t>((size_t)p->ntiles);
    p->carry_ml = cv.take<float2>((size_t)p->ntiles);
    p->carry_val = cv.take<float>((size_t)p->ntiles * p->F);
    p->gw = cv.take<float>((size_t)p->n_dst + 1);            // lse of every row as stored by the tile it ends in
    return cv.off;
}

}  // namespace tiga

using namespace tiga;

extern "C" size_t tiga_csr_attention_workspace_bytes(const tiga_csr* g, int32_t D) {
    if (attention_check(g, D) != TIGA_OK) return 0;
    CsrParams p{};
    p.n_dst = g->n_dst; p.n_edges = g->n_edges; p.n_src = g->n_src; p.F = D;
    p.ntiles = (g->n_dst + g->n_edges + CSR_TILE_ATT - 1) / CSR_TILE_ATT;
    return attention_carve(&p, nullptr) + 256;
}

extern "C" tiga_status tiga_apply_csr_attention(const tiga_csr* g, const float* q, const float* key, const float* value,
                                                int32_t D, float scale, float* out, float* lse,
                                                void* ws, size_t ws_bytes, void* stream) {
    tiga_status st = attention_check(g, D);
    if (st != TIGA_OK) return st;
    if (!isfinite(scale)) return TIGA_ERR_INVALID_ARG;
    if (g->n_dst == 0) return TIGA_OK;
    if (!g->rowptr || !aligned16(g->rowptr) || (g->n_edges > 0 && (!g->col || !aligned16(g->col)))) return TIGA_ERR_INVALID_ARG;
    if (!q || !out || !aligned16(q) || !aligned16(out)) return TIGA_ERR_INVALID_ARG;
    if (g->n_edges > 0 && (!key || !value || !aligned16(key) || !aligned16(value))) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_csr_attention_workspace_bytes(g, D)) return TIGA_ERR_WORKSPACE;
    CsrParams p{};
    p.rowptr = g->rowptr; p.col = g->col; p.w = nullptr;
    p.n_dst = g->n_dst; p.n_edges = g->n_edges; p.n_src = g->n_src; p.F = D; p.nvec = D / 4;
    p.ntiles = (g->n_dst + g->n_edges + CSR_TILE_ATT - 1) / CSR_TILE_ATT;
    p.q = q; p.key = key; p.x = value; p.scale = scale; p.out = out; p.lse = lse;
    attention_carve(&p, ws);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return g->rowptr_type == TIGA_I64 ? launch_attention<int64_t>(p, s) : launch_attention<int32_t>(p, s);
}

namespace tiga { unsigned check_status_csr_attention(bool reset) { return read_check_status(reset); } }
