// Stored-relation gf.apply for sm_100a: gather / message / reduce over a destination-
// oriented CSR (paper Sections 3.1, 4.2, 4.3) and its reverse mode (Section 5).
//
// Schedule (ours, not the paper's bounded-ragged Triton tile of Section 4.4):
//   * The merged sequence "row ends + edges" (N + E items) is cut into equal tiles, one CTA
//     per tile, so neither a 69k-edge row nor a run of a million empty rows unbalances a CTA
//     (a long row is split into partial states that are merged in edge order, the obligation
//     Section 4.4 attaches to splitting high-degree rows).
//   * A CTA stages its slice of rowptr, col and w in shared memory with coalesced streaming
//     loads, then splits its edges evenly over "workers" of G lanes.  A worker walks its edge
//     span in order; each lane owns 16 bytes of the feature row, so one gathered source row
//     is one fully coalesced 128-bit-per-lane request.  Several gathers are kept in flight
//     per lane.  The reducer state lives in registers.
//   * Rows wholly inside one worker's span are stored straight to global memory.  Partial
//     states (head / tail of a span) go to shared memory and are merged in edge order; the
//     CTA's trailing unfinished row becomes one carry-out in the workspace, which a small
//     fix-up kernel folds into the row, again in edge order.  No atomics in the forward, so
//     results are reproducible.
#include "csr_shared.cuh"
#include <atomic>
#include <mutex>

namespace tiga {

static std::atomic<long long> g_kernel_launches{0};
void note_launch() { g_kernel_launches.fetch_add(1, std::memory_order_relaxed); }

// --------------------------------------------------------------------------------------------
// Forward.  G lanes per worker, VPL 16-byte vectors per lane, RED = 0 sum / 1 max / 2 max whose
// edge positions are 64 bits wide (relations of 2^31 edges or more).
// --------------------------------------------------------------------------------------------
template <int RED> struct ArgOf { using type = int; };
template <> struct ArgOf<2> { using type = long long; };
template <int RED> using ArgT = typename ArgOf<RED>::type;

// 16-byte (32-bit positions) or 2 x 16-byte (64-bit positions) store of four edge positions
__device__ __forceinline__ void store_arg4(int* dst, int a0, int a1, int a2, int a3) {
    st_stream(reinterpret_cast<int4*>(dst), make_int4(a0, a1, a2, a3));
}
__device__ __forceinline__ void store_arg4(long long* dst, long long a0, long long a1, long long a2, long long a3) {
    st_stream(reinterpret_cast<longlong2*>(dst), make_longlong2(a0, a1));
    st_stream(reinterpret_cast<longlong2*>(dst + 2), make_longlong2(a2, a3));
}

template <int RED, int VPL, int VW>
struct State {
    using AT = ArgT<RED>;
    float v[VPL][VW];
    AT a[RED ? VPL : 1][RED ? VW : 1];
    __device__ __forceinline__ void reset() {
#pragma unroll
        for (int i = 0; i < VPL; ++i)
#pragma unroll
            for (int k = 0; k < VW; ++k) {
                // max: the empty state holds NaN, which every first message replaces through the
                // "greater or unordered" comparison below; stores turn a still-empty entry into 0
                v[i][k] = RED != 0 ? __int_as_float(0x7fc00000) : 0.f;
                if constexpr (RED != 0) a[i][k] = -1;
            }
    }
    // the value an entry is stored with (finalize: the empty state of max becomes 0)
    __device__ __forceinline__ float out(int i, int k) const {
        if constexpr (RED != 0) return a[i][k] < 0 ? 0.f : v[i][k];
        else return v[i][k];
    }
    // fold a message that comes later in edge order
    __device__ __forceinline__ void message(int i, int k, float wgt, float xv, AT e) {
        if constexpr (RED == 0) {
            v[i][k] = fmaf(wgt, xv, v[i][k]);
        } else {
            const float m = __fmul_rn(wgt, xv);        // one rounding, never contracted
            if (!(m <= v[i][k])) { v[i][k] = m; a[i][k] = e; }      // strictly greater, or the state is still empty
        }
    }
    // fold a partial state that comes later in edge order
    __device__ __forceinline__ void merge(int i, int k, float ov, AT oa) {
        if constexpr (RED == 0) {
            v[i][k] += ov;
        } else {
            if (oa >= 0 && !(ov <= v[i][k])) { v[i][k] = ov; a[i][k] = oa; }
        }
    }
};

// acc += w * x for two neighbouring features with one packed fused multiply-add (sm_100: one issue slot
// for both lanes of the pair; each half rounds once, exactly like fmaf)
__device__ __forceinline__ void fma_pair(float& a0, float& a1, float w, float x0, float x1) {
    unsigned long long acc, xx, ww;
    asm("mov.b64 %0, {%1, %2};" : "=l"(acc) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(xx) : "f"(x0), "f"(x1));
    asm("mov.b64 %0, {%1, %1};" : "=l"(ww) : "f"(w));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(ww), "l"(xx));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc));
}

// EXACT: the feature row fills the worker exactly (nvec == G * VPL): row stride and lane activity
// are compile-time constants, which removes address arithmetic and predicates from the edge loop.
template <typename XT, int G, int VPL, int RED, typename IT, bool EXACT>
__global__ void __launch_bounds__(CSR_THREADS, 5) csr_forward_kernel(const CsrParams p) {
    constexpr int VW = XTraits<XT>::VW;
    constexpr int NW = CSR_THREADS / G;          // workers per CTA
    constexpr int LV = G * VPL * VW;             // floats of one partial state
    constexpr int U = (VPL == 1) ? 4 : (VPL == 2 ? 2 : 1);   // gathers in flight per lane

    constexpr int TILE = RED == 0 ? CSR_TILE : CSR_TILE_MAX;
    __shared__ int s_ptr[TILE + 2];
    __shared__ __align__(16) int s_col[TILE + CSR_PAD];
    __shared__ __align__(16) float s_w[TILE + CSR_PAD];
    __shared__ long long s_coord[2];
    __shared__ int s_tag[2 * NW];                // local row of head (even) / tail (odd) partial, -1 = none
    __shared__ unsigned char s_first[NW];        // tail partial starts its chain
    extern __shared__ __align__(16) unsigned char s_dyn[];
    float* s_pv = reinterpret_cast<float*>(s_dyn);              // [2*NW][LV]
    using AT = ArgT<RED>;
    AT* s_pa = reinterpret_cast<AT*>(s_pv + 2 * NW * LV);       // [2*NW][LV] (max only; 2*NW*LV floats keep it 8-byte aligned)

    const Tile t = stage_tile<IT, false, TILE>(p, s_ptr, s_col, s_w, s_coord);
    const int wk = threadIdx.x / G;
    const int ln = threadIdx.x % G;
    const uint4* __restrict__ xlane = static_cast<const uint4*>(p.x) + ln;
    const unsigned nvec = EXACT ? (unsigned)(G * VPL) : (unsigned)p.nvec;
    const int F = EXACT ? G * VPL * VW : p.F;
    const long long e0 = t.e0;

    bool act[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) act[i] = EXACT ? true : (i * G + ln) < p.nvec;

    auto store_row = [&](long long row, const State<RED, VPL, VW>& s) {
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            if (!act[i]) continue;
            float* o = p.out + row * F + (size_t)(i * G + ln) * VW;
#pragma unroll
            for (int k = 0; k < VW; k += 4)
                st_stream(reinterpret_cast<float4*>(o + k), make_float4(s.out(i, k), s.out(i, k + 1), s.out(i, k + 2), s.out(i, k + 3)));
            if constexpr (RED != 0) {
                AT* ao = static_cast<AT*>(p.arg) + row * F + (size_t)(i * G + ln) * VW;
#pragma unroll
                for (int k = 0; k < VW; k += 4) store_arg4(ao + k, s.a[i][k], s.a[i][k + 1], s.a[i][k + 2], s.a[i][k + 3]);
            }
        }
    };
    auto store_partial = [&](int entry, const State<RED, VPL, VW>& s) {
#pragma unroll
        for (int i = 0; i < VPL; ++i)
#pragma unroll
            for (int k = 0; k < VW; ++k) {
                s_pv[entry * LV + (i * G + ln) * VW + k] = s.v[i][k];
                if constexpr (RED != 0) s_pa[entry * LV + (i * G + ln) * VW + k] = s.a[i][k];
            }
    };
    auto merge_partial = [&](int entry, State<RED, VPL, VW>& s) {
#pragma unroll
        for (int i = 0; i < VPL; ++i)
#pragma unroll
            for (int k = 0; k < VW; ++k)
                s.merge(i, k, s_pv[entry * LV + (i * G + ln) * VW + k],
                        RED ? s_pa[entry * LV + (i * G + ln) * VW + k] : AT(0));
    };

    // rows that end in this tile without an edge in it: the reducer identity (finalised to 0)
    {
        State<RED, VPL, VW> idn;
        idn.reset();
        for (int k = wk; k < t.nfin; k += NW) {
            const int ls = s_ptr[k] < 0 ? 0 : s_ptr[k];
            if (s_ptr[k + 1] == ls) store_row(t.i0 + k, idn);
        }
    }

    if (ln == 0) { s_tag[2 * wk] = -1; s_tag[2 * wk + 1] = -1; s_first[wk] = 0; }
    if (threadIdx.x == 0) p.carry_row[blockIdx.x] = -1;

    // spans start on multiples of U, so a step's U indices and weights are one vector load each
    const int chunk = ((t.ne + NW - 1) / NW + U - 1) / U * U;
    const int a = wk * chunk;
    const int b = (a + chunk < t.ne) ? a + chunk : t.ne;

    State<RED, VPL, VW> st;
    st.reset();
    int r = 0;
    bool tail_valid = false, tail_first = false;
    if (a < b) {
        r = row_of_edge(s_ptr, t.nrows, a);
        int cur_end = s_ptr[r + 1];
        bool head = (s_ptr[r] < 0 ? 0 : s_ptr[r]) < a;   // the row began in an earlier span of this tile
        for (int e = a; e < b; e += U) {
            uint4 xv[U][VPL];
            float wv[U];
            int cv[U];
            // entries past the span are readable (next worker's edges or the pad) and never used
            if constexpr (U == 4) {
                const int4 c4 = *reinterpret_cast<const int4*>(s_col + e);
                const float4 w4 = *reinterpret_cast<const float4*>(s_w + e);
                cv[0] = c4.x; cv[1] = c4.y; cv[2] = c4.z; cv[3] = c4.w;
                wv[0] = w4.x; wv[1] = w4.y; wv[2] = w4.z; wv[3] = w4.w;
            } else if constexpr (U == 2) {
                const int2 c2 = *reinterpret_cast<const int2*>(s_col + e);
                const float2 w2 = *reinterpret_cast<const float2*>(s_w + e);
                cv[0] = c2.x; cv[1] = c2.y; wv[0] = w2.x; wv[1] = w2.y;
            } else {
                cv[0] = s_col[e]; wv[0] = s_w[e];
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const unsigned c = (unsigned)cv[u];
                const uint4* src = xlane + (unsigned long long)c * nvec;      // one 32 x 32 -> 64 multiply
#pragma unroll
                for (int i = 0; i < VPL; ++i)
                    xv[u][i] = act[i] ? __ldg(src + i * G) : make_uint4(0, 0, 0, 0);
            }
            if (e + U <= b && e + U <= cur_end) {
                // common case: the whole batch lies inside the current row and the span
                constexpr bool PACKED = RED == 0 && sizeof(XT) == 4;
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float xf[VW];
#pragma unroll
                    for (int i = 0; i < VPL; ++i) {
                        XTraits<XT>::unpack(xv[u][i], xf);
                        if constexpr (PACKED) {
#pragma unroll
                            for (int k = 0; k < VW; k += 2) fma_pair(st.v[i][k], st.v[i][k + 1], wv[u], xf[k], xf[k + 1]);
                        } else {
#pragma unroll
                            for (int k = 0; k < VW; ++k) st.message(i, k, wv[u], xf[k], (AT)(e0 + e + u));
                        }
                    }
                }
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
                    }
                    float xf[VW];
#pragma unroll
                    for (int i = 0; i < VPL; ++i) {
                        XTraits<XT>::unpack(xv[u][i], xf);
#pragma unroll
                        for (int k = 0; k < VW; ++k) st.message(i, k, wv[u], xf[k], (AT)(e0 + e + u));
                    }
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

    // merge chains of partial states in edge order; the worker that opens a chain owns it
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
            if (ln == 0) p.carry_row[blockIdx.x] = (int32_t)(t.i0 + r);
#pragma unroll
            for (int i = 0; i < VPL; ++i) {
                if (!act[i]) continue;
                const size_t o = (size_t)blockIdx.x * F + (size_t)(i * G + ln) * VW;
#pragma unroll
                for (int k = 0; k < VW; ++k) {
                    p.carry_val[o + k] = st.v[i][k];
                    if constexpr (RED != 0) static_cast<AT*>(p.carry_arg)[o + k] = st.a[i][k];
                }
            }
        }
    }
}

// --------------------------------------------------------------------------------------------
// Forward for narrow rows (one or two 16-byte vectors per feature row, e.g. F = 8 fp16).
// A worker of G lanes would leave most of a warp idle here and a feature row is a single
// 128-bit load, so the work is split by ROW CLASS instead.  Every thread looks at one row
// (a warp at 32 consecutive rows):
//   * rows of at most ROW_OWN edges are summed by their own lane, in edge order (empty rows cost
//     one zero store; all 32 results of a warp leave as one contiguous kilobyte for F = 8);
//   * rows of up to ROW_GROUP edges are queued in shared memory and taken by GROUPS of eight lanes,
//     four rows per warp at a time: lanes stride over the row's edges, then the eight partial states
//     are combined by a halving exchange that leaves every lane with its share of the row's result,
//     so the row is stored by the group as one coalesced request;
//   * rows of up to ROW_HUGE edges are queued for whole warps (coalesced index loads, 128-bit
//     gathers, the same exchange over 32 lanes);
//   * rows above ROW_HUGE edges are cut into ROW_HUGE-edge chunks that are queued in the
//     workspace; a second kernel gives every chunk to a warp, a third folds the chunk states
//     of a row in order.
// The summation tree of every class is fixed, so results are reproducible (for max the tie rule
// "lowest edge position" makes the merge order irrelevant).
// --------------------------------------------------------------------------------------------
constexpr int ROW_OWN = 4;
constexpr int ROW_GROUP = 64;
constexpr int ROW_HUGE = 1024;       // longest row a single warp sums (the host lowers it for small relations: p.row_huge)
constexpr int ROW_HUGE_SMALL = 256;
constexpr int GROUP_LANES = 8;
constexpr int ROW_THREADS = 256;     // rows (= threads) per CTA of the row-class kernel

// Where a source row lives.  HOT (planned apply): col values below n_hot address the compact copy of the
// hot source rows, the others (minus n_hot) the feature table; both bases are set up once per thread.
template <bool HOT>
struct Sources {
    const uint4* cold;
    const uint4* hot;
    unsigned n_hot, nvec;
    long long n_all;              // checked build: range of the indices
    __device__ __forceinline__ explicit Sources(const CsrParams& p) {
        nvec = (unsigned)p.nvec;
        n_all = p.n_src;
        n_hot = HOT ? (unsigned)p.n_hot : 0u;
        cold = static_cast<const uint4*>(p.x) - (size_t)n_hot * nvec;
        hot = HOT ? static_cast<const uint4*>(p.x_hot) : cold;
    }
    __device__ __forceinline__ const uint4* row(unsigned c) const {
        c = checked(c, n_all, CHECK_SOURCE);
        const uint4* base = (HOT && c < n_hot) ? hot : cold;
        return base + (unsigned long long)c * nvec;          // one 32 x 32 -> 64 multiply
    }
};

// Combines the states of the L lanes of an aligned group by a halving exchange: at every step a lane
// sends the half of its values that its partner keeps and folds the partner's half into its own, so
// the number of values per lane halves while the number of lanes summed doubles; once one value is
// left the remaining steps are plain butterflies.  Afterwards lane gl of the group holds, in its first
// kept<C, L>() entries, the group totals of the values starting at spread_index<NVAL, L>(gl).
template <int RED, int C, int J, int L>
struct Spread {
    static __device__ __forceinline__ void run(float* v, ArgT<RED>* a, int gl) {
        using AT = ArgT<RED>;
        if constexpr ((1 << J) < L) {
            constexpr int o = 1 << J;
            constexpr unsigned FULL = 0xffffffffu;
            if constexpr (C > 1) {
                constexpr int H = C / 2;
                const bool up = (gl & o) != 0;
#pragma unroll
                for (int k = 0; k < H; ++k) {
                    const float send = up ? v[k] : v[k + H];
                    const float keep = up ? v[k + H] : v[k];
                    const float got = __shfl_xor_sync(FULL, send, o);
                    if constexpr (RED == 0) {
                        v[k] = keep + got;
                    } else {
                        const AT sa = up ? a[k] : a[k + H];
                        const AT ka = up ? a[k + H] : a[k];
                        const AT ga = __shfl_xor_sync(FULL, sa, o);
                        // larger message wins; equal messages: the lower edge position
                        const bool take = ga >= 0 && (ka < 0 || got > keep || (got == keep && ga < ka));
                        v[k] = take ? got : keep;
                        a[k] = take ? ga : ka;
                    }
                }
                Spread<RED, H, J + 1, L>::run(v, a, gl);
            } else {
                const float got = __shfl_xor_sync(FULL, v[0], o);
                if constexpr (RED == 0) {
                    v[0] += got;
                } else {
                    const AT ga = __shfl_xor_sync(FULL, a[0], o);
                    const bool take = ga >= 0 && (a[0] < 0 || got > v[0] || (got == v[0] && ga < a[0]));
                    if (take) { v[0] = got; a[0] = ga; }
                }
                Spread<RED, 1, J + 1, L>::run(v, a, gl);
            }
        }
    }
};

template <int NVAL, int L>
__device__ __forceinline__ int spread_index(int gl) {
    int base = 0;
#pragma unroll
    for (int j = 0; (1 << j) < L && (NVAL >> j) > 1; ++j) base += ((gl >> j) & 1) * (NVAL >> (j + 1));
    return base;
}

// lanes of the group stride over edges [es, es + n) of one row; every lane returns its partial state.
// W: the relation has edge weights (otherwise every message is the source row itself).  The indices of
// the next step are requested before the gathers of the current one are consumed, so an index load and
// a gather are in flight at the same time instead of one after the other.
template <typename XT, int NV, int RED, int L, int UNR, bool HOT, bool W>
__device__ __forceinline__ State<RED, NV, XTraits<XT>::VW> strided_row(const CsrParams& p, const Sources<HOT>& src, long long es, int n, int gl) {
    constexpr int VW = XTraits<XT>::VW;
    State<RED, NV, VW> s;
    s.reset();
    const int32_t* __restrict__ colp = p.col + es;
    const float* __restrict__ wp = W ? p.w + es : nullptr;
    unsigned cn[UNR];
    float wn[UNR];
    auto fetch = [&](int k) {
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int idx = k + L * u;
            const int at = idx < n ? idx : (k < n ? k : 0);
            cn[u] = n > 0 ? (unsigned)ld_stream(colp + at) : 0u;
            wn[u] = (W && n > 0) ? ld_stream(wp + at) : 1.f;
        }
    };
    fetch(gl);
    for (int k = gl; k < n; k += L * UNR) {
        uint4 xv[UNR][NV];
        float wv[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const bool in = k + L * u < n;
            wv[u] = wn[u];
            const uint4* r = src.row(cn[u]);
#pragma unroll
            for (int i = 0; i < NV; ++i) xv[u][i] = in ? __ldg(r + i) : make_uint4(0, 0, 0, 0);
        }
        if (k + L * UNR < n) fetch(k + L * UNR);
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            if (k + L * u < n) {
                if constexpr (RED == 0 && !W) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) XTraits<XT>::add_to(xv[u][i], &s.v[i][0]);
                } else {
                    float xf[VW];
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        XTraits<XT>::unpack(xv[u][i], xf);
#pragma unroll
                        for (int q = 0; q < VW; ++q) s.message(i, q, wv[u], xf[q], (ArgT<RED>)(es + k + L * u));
                    }
                }
            }
        }
    }
    return s;
}

template <typename XT, int NV, int RED>
__device__ __forceinline__ void store_state(const CsrParams& p, float* out, ArgT<RED>* arg, const State<RED, NV, XTraits<XT>::VW>& s) {
    constexpr int VW = XTraits<XT>::VW;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
#pragma unroll
        for (int k = 0; k < VW; k += 4) {
            st_stream(reinterpret_cast<float4*>(out + i * VW + k), make_float4(s.out(i, k), s.out(i, k + 1), s.out(i, k + 2), s.out(i, k + 3)));
            if constexpr (RED != 0) store_arg4(arg + i * VW + k, s.a[i][k], s.a[i][k + 1], s.a[i][k + 2], s.a[i][k + 3]);
        }
    }
}

// combine the partial states of a group of L lanes and store the row: every lane writes its share
template <typename XT, int NV, int RED, int L>
__device__ __forceinline__ void reduce_and_store(State<RED, NV, XTraits<XT>::VW>& s, int gl, bool valid, float* out, ArgT<RED>* arg) {
    constexpr int NVAL = NV * XTraits<XT>::VW;
    constexpr int KEEP = NVAL >= L ? NVAL / L : 1;
    float* v = &s.v[0][0];
    ArgT<RED>* a = &s.a[0][0];
    Spread<RED, NVAL, 0, L>::run(v, a, gl);
    if (valid && gl < NVAL) {
        const int base = spread_index<NVAL, L>(gl);
#pragma unroll
        for (int k = 0; k < KEEP; ++k) {
            st_stream(out + base + k, v[k]);
            if constexpr (RED != 0) st_stream(arg + base + k, a[k]);
        }
    }
}

template <typename XT, int NV, int RED, typename IT, bool HOT, bool W>
__global__ void __launch_bounds__(ROW_THREADS, 1536 / ROW_THREADS) csr_rows_kernel(const CsrParams p) {
    constexpr int VW = XTraits<XT>::VW;
    constexpr unsigned FULL = 0xffffffffu;
    using St = State<RED, NV, VW>;
    const IT* __restrict__ rowptr = static_cast<const IT*>(p.rowptr);
    const Sources<HOT> src(p);
    const int lane = threadIdx.x & 31;
    const long long row = ((long long)blockIdx.x * ROW_THREADS + threadIdx.x);      // warp-contiguous rows
    const bool valid = row < p.n_dst;
    const long long es = valid ? (long long)rowptr[row] : 0;
    const long long ee = valid ? (long long)rowptr[row + 1] : 0;
    const long long deg = ee - es;

    // queues of the CTA's longer rows: group rows fill from the front, warp rows from the back
    __shared__ short q_row[ROW_THREADS];
    __shared__ long long q_start[ROW_THREADS];
    __shared__ int q_len[ROW_THREADS];
    __shared__ int q_ng, q_nw, q_next;
    if (threadIdx.x == 0) { q_ng = 0; q_nw = 0; q_next = 0; }
    __syncthreads();
    const bool is_g = valid && deg > ROW_OWN && deg <= ROW_GROUP;
    const bool is_w = valid && deg > ROW_GROUP && deg <= p.row_huge;
    {
        const unsigned mg = __ballot_sync(FULL, is_g), mw = __ballot_sync(FULL, is_w);
        int bg = 0, bw = 0;
        if (lane == 0) {
            if (mg) bg = atomicAdd(&q_ng, __popc(mg));
            if (mw) bw = atomicAdd(&q_nw, __popc(mw));
        }
        bg = __shfl_sync(FULL, bg, 0); bw = __shfl_sync(FULL, bw, 0);
        const unsigned lt = (1u << lane) - 1u;
        if (is_g || is_w) {
            const int slot = is_g ? bg + __popc(mg & lt) : ROW_THREADS - 1 - (bw + __popc(mw & lt));
            q_row[slot] = (short)threadIdx.x; q_start[slot] = es; q_len[slot] = (int)deg;
        }
    }

    // short rows: one lane each, edge order, one pass with all gathers in flight
    St st;
    st.reset();
    if (valid && deg <= ROW_OWN) {
        const int n = (int)deg;
        uint4 xv[ROW_OWN][NV];
        float wv[ROW_OWN];
#pragma unroll
        for (int u = 0; u < ROW_OWN; ++u) {
            const bool in = u < n;
            const long long e = es + (in ? u : 0);
            const unsigned c = in ? (unsigned)__ldg(p.col + e) : 0u;
            wv[u] = (W && in) ? __ldg(p.w + e) : 1.f;
            const uint4* r = src.row(c);
#pragma unroll
            for (int i = 0; i < NV; ++i) xv[u][i] = in ? __ldg(r + i) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < ROW_OWN; ++u) {
            if (u < n) {
                if constexpr (RED == 0 && !W) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) XTraits<XT>::add_to(xv[u][i], &st.v[i][0]);
                } else {
                    float xf[VW];
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        XTraits<XT>::unpack(xv[u][i], xf);
#pragma unroll
                        for (int q = 0; q < VW; ++q) st.message(i, q, wv[u], xf[q], (ArgT<RED>)(es + u));
                    }
                }
            }
        }
        store_state<XT, NV, RED>(p, p.out + row * p.F, RED ? static_cast<ArgT<RED>*>(p.arg) + row * p.F : nullptr, st);
    }
    __syncthreads();
    const long long row0 = (long long)blockIdx.x * ROW_THREADS;
    const int ng = q_ng, nw = q_nw;

    // rows for groups of eight lanes: 32 groups per CTA, four rows per warp at a time
    {
        const int gl = lane & (GROUP_LANES - 1);
        const int gid = (threadIdx.x >> 5) * (32 / GROUP_LANES) + lane / GROUP_LANES;
        constexpr int NGROUPS = ROW_THREADS / GROUP_LANES;
        for (int it0 = 0; it0 < ng; it0 += NGROUPS) {           // uniform over the CTA
            const int it = it0 + gid;
            const bool have = it < ng;
            const long long rs = have ? q_start[it] : 0;
            const int rn = have ? q_len[it] : 0;
            const long long r = row0 + (have ? q_row[it] : 0);
            St part = strided_row<XT, NV, RED, GROUP_LANES, 4, HOT, W>(p, src, rs, rn, gl);
            __syncwarp();
            reduce_and_store<XT, NV, RED, GROUP_LANES>(part, gl, have, p.out + r * p.F, RED ? static_cast<ArgT<RED>*>(p.arg) + r * p.F : nullptr);
        }
    }
    // rows for whole warps, taken from the back of the queue
    for (;;) {
        int idx = 0;
        if (lane == 0) idx = atomicAdd(&q_next, 1);
        idx = __shfl_sync(FULL, idx, 0);
        if (idx >= nw) break;
        const int slot = ROW_THREADS - 1 - idx;
        const long long r = row0 + q_row[slot];
        St part = strided_row<XT, NV, RED, 32, 4, HOT, W>(p, src, q_start[slot], q_len[slot], lane);
        reduce_and_store<XT, NV, RED, 32>(part, lane, true, p.out + r * p.F, RED ? static_cast<ArgT<RED>*>(p.arg) + r * p.F : nullptr);
    }
    // huge rows: queue their chunks
    if (valid && deg > p.row_huge) {
        const int chunks = (int)((deg + p.row_huge - 1) / p.row_huge);
        const int base = atomicAdd(p.huge_count, chunks);
        for (int c = 0; c < chunks; ++c) p.huge_list[base + c] = make_int4((int)row, c, chunks, base);
    }
}

// one warp per queued chunk of a huge row
template <typename XT, int NV, int RED, typename IT, bool HOT, bool W>
__global__ void __launch_bounds__(CSR_THREADS) csr_huge_chunks_kernel(const CsrParams p) {
    const IT* __restrict__ rowptr = static_cast<const IT*>(p.rowptr);
    const Sources<HOT> src(p);
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * (CSR_THREADS / 32);
    const int total = *p.huge_count;
    for (int idx = blockIdx.x * (CSR_THREADS / 32) + (threadIdx.x >> 5); idx < total; idx += nwarps) {
        const int4 ent = p.huge_list[idx];
        const long long es = (long long)rowptr[ent.x] + (long long)ent.y * p.row_huge;
        const long long ee = (long long)rowptr[ent.x + 1];
        const int n = (int)(ee - es < p.row_huge ? ee - es : p.row_huge);
        auto part = strided_row<XT, NV, RED, 32, 8, HOT, W>(p, src, es, n, lane);
        reduce_and_store<XT, NV, RED, 32>(part, lane, true, p.carry_val + (size_t)idx * p.F, RED ? static_cast<ArgT<RED>*>(p.carry_arg) + (size_t)idx * p.F : nullptr);
    }
}

// fold the chunk states of every huge row in chunk (= edge) order; one thread per (row, feature)
template <int RED>
__global__ void csr_huge_fold_kernel(const CsrParams p) {
    const int total = *p.huge_count;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < (long long)total * p.F; t += nthreads) {
        const int idx = (int)(t / p.F), f = (int)(t % p.F);
        const int4 ent = p.huge_list[idx];
        if (ent.y != 0) continue;
        float v = p.carry_val[(size_t)idx * p.F + f];
        using AT = ArgT<RED>;
        const AT* carg = static_cast<const AT*>(p.carry_arg);
        AT a = RED ? carg[(size_t)idx * p.F + f] : AT(0);
        for (int c = 1; c < ent.z; ++c) {
            const float ov = p.carry_val[(size_t)(idx + c) * p.F + f];
            if (RED == 0) v += ov;
            else {
                const AT oa = carg[(size_t)(idx + c) * p.F + f];
                if (oa >= 0 && (a < 0 || ov > v)) { v = ov; a = oa; }
            }
        }
        p.out[(size_t)ent.x * p.F + f] = v;
        if (RED) static_cast<AT*>(p.arg)[(size_t)ent.x * p.F + f] = a;
    }
}

// Fold the carry-outs of consecutive tiles that belong to one row into that row, in edge
// order.  One thread per (tile, feature); only the first tile of a run does the work.
template <int RED>
__global__ void csr_fixup_kernel(const CsrParams p) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long tile = idx / p.F;
    const int f = (int)(idx % p.F);
    if (tile >= p.ntiles) return;
    const int row = p.carry_row[tile];
    if (row < 0) return;
    if (tile > 0 && p.carry_row[tile - 1] == row) return;
    float v = p.carry_val[tile * p.F + f];
    using AT = ArgT<RED>;
    const AT* carg = static_cast<const AT*>(p.carry_arg);
    AT a = RED ? carg[tile * p.F + f] : AT(0);
    for (long long u = tile + 1; u < p.ntiles && p.carry_row[u] == row; ++u) {
        const float ov = p.carry_val[u * p.F + f];
        if (RED == 0) v += ov;
        else {
            const AT oa = carg[u * p.F + f];
            if (oa >= 0 && (a < 0 || ov > v)) { v = ov; a = oa; }
        }
    }
    const size_t o = (size_t)row * p.F + f;
    if (RED == 0) {
        p.out[o] = v + p.out[o];
    } else {
        const float ov = p.out[o];
        const AT oa = static_cast<AT*>(p.arg)[o];
        if (oa >= 0 && (a < 0 || ov > v)) { v = ov; a = oa; }
        p.out[o] = v;
        static_cast<AT*>(p.arg)[o] = a;
    }
}

// --------------------------------------------------------------------------------------------
// Backward, sum reducer (Section 5).  Same tiles and workers; every edge is independent:
//   gw[e] = x[col[e],:] . gy[row,:]            (one value per edge position, duplicates not merged)
//   gx[col[e],:] += w[e] * gy[row,:]           (reverse incidence: vector atomics)
// --------------------------------------------------------------------------------------------
// four consecutive features of a source row as fp32: one 128-bit load (fp32 rows) or one 64-bit load (fp16 rows)
template <typename XT>
__device__ __forceinline__ float4 load_x4(const void* x, unsigned long long vec) {
    if constexpr (sizeof(XT) == 4) {
        return __ldg(static_cast<const float4*>(x) + vec);
    } else {
        const uint2 raw = __ldg(static_cast<const uint2*>(x) + vec);
        const float2 lo = __half22float2(*reinterpret_cast<const __half2*>(&raw.x));
        const float2 hi = __half22float2(*reinterpret_cast<const __half2*>(&raw.y));
        return make_float4(lo.x, lo.y, hi.x, hi.y);
    }
}

template <int G, int VPL, typename IT, typename XT>
__global__ void __launch_bounds__(CSR_THREADS) csr_backward_sum_kernel(const CsrParams p) {
    constexpr int NW = CSR_THREADS / G;
    constexpr int U = (VPL == 1) ? 4 : (VPL == 2 ? 2 : 1);
    constexpr int TILE = CSR_TILE_BWD;
    __shared__ int s_ptr[TILE + 2];
    __shared__ int s_col[TILE + CSR_PAD];
    __shared__ float s_w[TILE + CSR_PAD];
    __shared__ float s_gw[TILE];
    __shared__ long long s_coord[2];

    const Tile t = stage_tile<IT, false, TILE>(p, s_ptr, s_col, s_w, s_coord);
    const int wk = threadIdx.x / G;
    const int ln = threadIdx.x % G;
    // lanes of one worker stay converged; workers of one warp do not
    const unsigned wmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) & ~(G - 1)));
    const float4* __restrict__ gybase = reinterpret_cast<const float4*>(p.gy);
    float4* gxlane = reinterpret_cast<float4*>(p.gx) + ln;
    const unsigned nvec = (unsigned)p.nvec;

    bool act[VPL];
#pragma unroll
    for (int i = 0; i < VPL; ++i) act[i] = (i * G + ln) < p.nvec;

    const int chunk = (t.ne + NW - 1) / NW;
    const int a = wk * chunk;
    const int b = (a + chunk < t.ne) ? a + chunk : t.ne;
    if (a < b) {
        int r = row_of_edge(s_ptr, t.nrows, a);
        int cur_end = s_ptr[r + 1];
        float4 g[VPL];
        auto load_gy = [&](int rr) {
#pragma unroll
            for (int i = 0; i < VPL; ++i)
                g[i] = act[i] ? __ldg(gybase + (t.i0 + rr) * p.nvec + i * G + ln) : make_float4(0.f, 0.f, 0.f, 0.f);
        };
        load_gy(r);
        for (int e = a; e < b; e += U) {
            float4 xv[U][VPL];
            int cv[U];
            float wv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                // entries past the span are readable (next worker's edges or the pad) and never used
                cv[u] = s_col[e + u];
                wv[u] = s_w[e + u];
                if (p.gw) {
#pragma unroll
                    for (int i = 0; i < VPL; ++i)
                        xv[u][i] = act[i] ? load_x4<XT>(p.x, (unsigned long long)(unsigned)cv[u] * nvec + i * G + ln) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (e + u < b) {           // uniform inside a worker
                    if (e + u >= cur_end) {
                        do { ++r; cur_end = s_ptr[r + 1]; } while (e + u >= cur_end);
                        load_gy(r);
                    }
                    if (p.gw) {
                        float d = 0.f;
#pragma unroll
                        for (int i = 0; i < VPL; ++i) {
                            d = fmaf(xv[u][i].x, g[i].x, d); d = fmaf(xv[u][i].y, g[i].y, d);
                            d = fmaf(xv[u][i].z, g[i].z, d); d = fmaf(xv[u][i].w, g[i].w, d);
                        }
#pragma unroll
                        for (int o = G / 2; o > 0; o >>= 1) d += __shfl_xor_sync(wmask, d, o, G);
                        if (ln == 0) s_gw[e + u] = d;
                    }
                    if (p.gx) {
#pragma unroll
                        for (int i = 0; i < VPL; ++i)
                            if (act[i])
                                atomicAdd(gxlane + (unsigned long long)(unsigned)cv[u] * nvec + i * G,
                                          make_float4(wv[u] * g[i].x, wv[u] * g[i].y, wv[u] * g[i].z, wv[u] * g[i].w));
                    }
                }
            }
        }
    }
    if (p.gw) {
        __syncthreads();
        for (int k = threadIdx.x; k < t.ne; k += CSR_THREADS) st_stream(p.gw + t.e0 + k, s_gw[k]);
    }
}

// Backward, max reducer: the cotangent of (i, f) goes through the selected edge only.
// One thread per four consecutive features of a row.  They often select the same edge (always, for a
// row with one edge): then the thread gathers the source row slice with one vector load, sends the
// feature gradient as one vector atomic and contributes one value to the edge gradient; a warp sums
// the edge-gradient contributions of such threads that share an edge (two rounds, each for the edge of
// the lowest lane not served yet; what is left goes out one by one: more rounds measured slower), so an
// edge receives one atomic instead of up to 32 on the same address.  Features whose selected edges
// differ go one by one.
template <typename XT, int RED>
__global__ void csr_backward_max_kernel(const CsrParams p) {
    using AT = ArgT<RED>;
    constexpr unsigned FULL = 0xffffffffu;
    const long long idx = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const int lane = threadIdx.x & 31;
    const bool in = idx < p.n_dst * p.F;
    AT a[4] = {AT(-1), AT(-1), AT(-1), AT(-1)};
    float g[4] = {0.f, 0.f, 0.f, 0.f};
    if (in) {
        const AT* ap = static_cast<const AT*>(p.arg) + idx;
        if constexpr (sizeof(AT) == 4) {
            const int4 v = *reinterpret_cast<const int4*>(ap);
            a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
        } else {
            const longlong2 v0 = *reinterpret_cast<const longlong2*>(ap), v1 = *reinterpret_cast<const longlong2*>(ap + 2);
            a[0] = v0.x; a[1] = v0.y; a[2] = v1.x; a[3] = v1.y;
        }
        const float4 gv = *reinterpret_cast<const float4*>(p.gy + idx);
        g[0] = gv.x; g[1] = gv.y; g[2] = gv.z; g[3] = gv.w;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            if (a[k] >= 0) a[k] = checked(a[k], p.n_edges, CHECK_EDGE);
    }
    const int f0 = (int)(idx % p.F);
    const bool uni = in && a[0] >= 0 && a[0] == a[1] && a[1] == a[2] && a[2] == a[3];
    const AT e = uni ? a[0] : AT(-1);
    float contrib = 0.f;
    if (uni) {
        const long long j = checked(p.col[e], p.n_src, CHECK_SOURCE);
        const float wgt = p.w ? p.w[e] : 1.f;
        if (p.gx) atomicAdd(reinterpret_cast<float4*>(p.gx + j * p.F + f0), make_float4(wgt * g[0], wgt * g[1], wgt * g[2], wgt * g[3]));
        if (p.gw) {
            const float4 xv = load_x4<XT>(p.x, (unsigned long long)(j * p.F + f0) >> 2);
            contrib = fmaf(xv.w, g[3], fmaf(xv.z, g[2], fmaf(xv.y, g[1], xv.x * g[0])));
        }
    } else if (in) {
        // the four chains (edge -> source -> feature) are independent: all loads of a level first
        long long j[4];
        float wv[4], xv[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const AT ek = a[k] >= 0 ? a[k] : AT(0);
            j[k] = checked(p.col[ek], p.n_src, CHECK_SOURCE);
            wv[k] = p.w ? p.w[ek] : 1.f;
        }
        if (p.gw) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if constexpr (sizeof(XT) == 4) xv[k] = static_cast<const float*>(p.x)[j[k] * p.F + f0 + k];
                else xv[k] = __half2float(static_cast<const __half*>(p.x)[j[k] * p.F + f0 + k]);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (a[k] < 0) continue;
            if (p.gx) atomicAdd(p.gx + j[k] * p.F + f0 + k, wv[k] * g[k]);
            if (p.gw) atomicAdd(p.gw + a[k], xv[k] * g[k]);
        }
    }
    if (!p.gw) return;
    unsigned remaining = __ballot_sync(FULL, uni);
    for (int round = 0; remaining; ++round) {           // warp uniform
        if (round == 2) {
            if ((remaining >> lane) & 1u) atomicAdd(p.gw + e, contrib);
            break;
        }
        const int leader = __ffs(remaining) - 1;
        const AT el = __shfl_sync(FULL, e, leader);
        const bool mine = uni && e == el;
        float s = mine ? contrib : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
        if (lane == leader) atomicAdd(p.gw + el, s);
        remaining &= ~__ballot_sync(FULL, mine);
    }
}

// The same with one thread per (i, f): more threads in flight and no serial work per thread, which is the
// faster form while the gradient table fits L2 (atomics at L2 speed); the host picks by the table's size.
template <typename XT, int RED>
__global__ void csr_backward_max_each_kernel(const CsrParams p) {
    using AT = ArgT<RED>;
    constexpr unsigned FULL = 0xffffffffu;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    AT e = idx < p.n_dst * p.F ? static_cast<const AT*>(p.arg)[idx] : AT(-1);
    if (e >= 0) e = checked(e, p.n_edges, CHECK_EDGE);
    const bool act = e >= 0;
    float contrib = 0.f;
    if (act) {
        const int f = (int)(idx % p.F);
        const long long j = checked(p.col[e], p.n_src, CHECK_SOURCE);
        const float g = p.gy[idx];
        if (p.gx) atomicAdd(p.gx + j * p.F + f, (p.w ? p.w[e] : 1.f) * g);
        if (p.gw) {
            float xv;
            if constexpr (sizeof(XT) == 4) xv = static_cast<const float*>(p.x)[j * p.F + f];
            else xv = __half2float(static_cast<const __half*>(p.x)[j * p.F + f]);
            contrib = xv * g;
        }
    }
    if (!p.gw) return;
    unsigned remaining = __ballot_sync(FULL, act);
    for (int round = 0; remaining; ++round) {           // warp uniform
        if (round == 2) {
            if ((remaining >> lane) & 1u) atomicAdd(p.gw + e, contrib);
            break;
        }
        const int leader = __ffs(remaining) - 1;
        const AT el = __shfl_sync(FULL, e, leader);
        const bool mine = act && e == el;
        float s = mine ? contrib : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
        if (lane == leader) atomicAdd(p.gw + el, s);
        remaining &= ~__ballot_sync(FULL, mine);
    }
}

// --------------------------------------------------------------------------------------------
// Degree histogram and validation
// --------------------------------------------------------------------------------------------
template <typename IT>
__global__ void __launch_bounds__(1024, 1) degree_hist_kernel(const IT* __restrict__ rowptr, long long n, int nbins,
                                                              unsigned long long* hist, unsigned long long* maxdeg) {
    extern __shared__ unsigned int s_hist[];
    constexpr unsigned FULL = 0xffffffffu;
    for (int k = threadIdx.x; k < nbins; k += blockDim.x) s_hist[k] = 0;
    __syncthreads();
    // Most rows of a skewed relation have a handful of edges: degrees below LOW are counted in registers
    // (no shared-memory atomics on a few hot bins) and folded in once per warp at the end.  The eight
    // counters are bytes of one 64-bit word (one shift and one add per row), emptied into full-width
    // counters before a byte can overflow.
    constexpr int LOW = 8, UNR = 8, FLUSH_STEPS = 248 / UNR;
    const bool low_ok = nbins > LOW + 1;
    const int lane = threadIdx.x & 31;
    unsigned long long packed = 0ull;
    int steps = 0;
    auto unpack = [&]() {
#pragma unroll
        for (int k = 0; k < LOW; ++k) {
            const unsigned tot = __reduce_add_sync(FULL, (unsigned)((packed >> (8 * k)) & 255ull));
            if (lane == 0 && tot) atomicAdd(&s_hist[k], tot);
        }
        packed = 0ull;
    };
    long long mx = 0;
    // A warp reads 32 consecutive row offsets with one coalesced load and forms 31 degrees from them (a lane's
    // row ends where its neighbour's begins; the last lane only supplies that end), so consecutive chunks
    // overlap by one offset.  All loads of a step are issued before any is used.
    const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long c0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; c0 * 31 < n; c0 += warps * UNR) {
        if (++steps == FLUSH_STEPS) { unpack(); steps = 0; }
        long long v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const long long i = (c0 + u * warps) * 31 + lane;
            v[u] = i <= n ? (long long)rowptr[i] : 0;
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const long long i = (c0 + u * warps) * 31 + lane;
            const long long d = __shfl_down_sync(FULL, v[u], 1) - v[u];
            if (lane == 31 || i >= n || d < 0) continue;
            mx = d > mx ? d : mx;
            if (low_ok && d < LOW) packed += 1ull << (8 * (int)d);
            else atomicAdd(&s_hist[d < nbins - 1 ? (int)d : nbins - 1], 1u);
        }
    }
    if (low_ok) unpack();
    for (int o = 16; o > 0; o >>= 1) {
        const long long other = __shfl_xor_sync(FULL, mx, o);
        mx = other > mx ? other : mx;
    }
    if (lane == 0 && mx > 0) atomicMax(maxdeg, (unsigned long long)mx);
    __syncthreads();
    for (int k = threadIdx.x; k < nbins; k += blockDim.x)
        if (s_hist[k]) atomicAdd(hist + k, (unsigned long long)s_hist[k]);
}

template <typename IT>
__global__ void validate_kernel(const IT* __restrict__ rowptr, const int32_t* __restrict__ col,
                                long long n_dst, long long n_src, long long n_edges, int* flags) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long t0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    int bad = 0;
    if (t0 == 0) {
        if ((long long)rowptr[0] != 0) bad |= 1;
        if ((long long)rowptr[n_dst] != n_edges) bad |= 2;
    }
    for (long long i = t0; i < n_dst; i += stride)
        if ((long long)rowptr[i + 1] < (long long)rowptr[i]) bad |= 4;
    for (long long e = t0; e < n_edges; e += stride) {
        const int c = col[e];
        if (c < 0 || (long long)c >= n_src) bad |= 8;
    }
    if (bad) atomicOr(flags, bad);
}

// --------------------------------------------------------------------------------------------
// Host side
// --------------------------------------------------------------------------------------------
static bool pick_shape(int nvec, int* G, int* VPL) {
    if (nvec <= 0) return false;
    if (nvec <= 32) {
        int g = 1;
        while (g < nvec) g <<= 1;
        *G = g; *VPL = 1;
        return true;
    }
    *G = 32;
    const int v = (nvec + 31) / 32;
    if (v <= 2) *VPL = 2; else if (v <= 4) *VPL = 4; else return false;
    return true;
}

// Chunk length of the row-class path: a row is summed by one warp up to this many edges.  On a small relation
// the longest row would otherwise be one warp's latency chain and set the time of the whole call (R-MAT,
// F = 8 fp16: 2^20 edges 0.137 -> 0.042 ms with 256 instead of 4096; 2^26 edges 0.45 -> 0.39 ms and 2^28 edges
// 1.61 -> 1.48 ms with 1024; 2^30 edges the same with 1024 and 4096).
static int row_huge_of(const tiga_csr* g) { return g->n_edges >= (1LL << 25) ? ROW_HUGE : ROW_HUGE_SMALL; }

// tiles of a relation for a given tile length; without one, for the shortest (sizes workspaces, bounds grids)
static long long num_tiles(const tiga_csr* g, int tile = CSR_TILE_MIN) { return (g->n_dst + g->n_edges + tile - 1) / tile; }

template <typename XT, int G, int VPL, int RED, typename IT>
static tiga_status launch_fwd_t(const CsrParams& p, cudaStream_t s) {
    constexpr int NW = CSR_THREADS / G;
    const size_t dyn = (size_t)2 * NW * G * VPL * XTraits<XT>::VW * (sizeof(float) + (RED ? sizeof(ArgT<RED>) : 0));
    auto kern = p.nvec == G * VPL ? csr_forward_kernel<XT, G, VPL, RED, IT, true> : csr_forward_kernel<XT, G, VPL, RED, IT, false>;
    if (dyn > 16 * 1024) TIGA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn));
    kern<<<counted((unsigned)p.ntiles), CSR_THREADS, dyn, s>>>(p);
    return launch_status();
}

// rows of at most two 16-byte vectors: row-class kernels; HOT serves the hot source rows from p.x_hot
template <typename XT, int NV, int RED, typename IT, bool HOT, bool W>
static tiga_status launch_fwd_narrow_t(const CsrParams& p, cudaStream_t s) {
    TIGA_CUDA_TRY(cudaMemsetAsync(p.huge_count, 0, sizeof(int), s));
    const unsigned blocks = (unsigned)((p.n_dst + ROW_THREADS - 1) / ROW_THREADS);
    csr_rows_kernel<XT, NV, RED, IT, HOT, W><<<counted(blocks), ROW_THREADS, 0, s>>>(p);
    csr_huge_chunks_kernel<XT, NV, RED, IT, HOT, W><<<counted(148 * 8), CSR_THREADS, 0, s>>>(p);
    csr_huge_fold_kernel<RED><<<counted(148 * 2), 256, 0, s>>>(p);
    return launch_status();
}

template <typename XT, int RED, typename IT, bool HOT>
static tiga_status launch_fwd_narrow(const CsrParams& p, cudaStream_t s) {
    if (p.nvec == 1) return p.w ? launch_fwd_narrow_t<XT, 1, RED, IT, HOT, true>(p, s) : launch_fwd_narrow_t<XT, 1, RED, IT, HOT, false>(p, s);
    return p.w ? launch_fwd_narrow_t<XT, 2, RED, IT, HOT, true>(p, s) : launch_fwd_narrow_t<XT, 2, RED, IT, HOT, false>(p, s);
}

template <typename XT, int RED, typename IT>
static tiga_status launch_fwd_g(const CsrParams& p, int G, int VPL, cudaStream_t s) {
    if (p.nvec <= 2) return launch_fwd_narrow<XT, RED, IT, false>(p, s);
    switch (G) {
        case 1: return launch_fwd_t<XT, 1, 1, RED, IT>(p, s);
        case 2: return launch_fwd_t<XT, 2, 1, RED, IT>(p, s);
        case 4: return launch_fwd_t<XT, 4, 1, RED, IT>(p, s);
        case 8: return launch_fwd_t<XT, 8, 1, RED, IT>(p, s);
        case 16: return launch_fwd_t<XT, 16, 1, RED, IT>(p, s);
        default:
            if (VPL == 1) return launch_fwd_t<XT, 32, 1, RED, IT>(p, s);
            if (VPL == 2) return launch_fwd_t<XT, 32, 2, RED, IT>(p, s);
            return launch_fwd_t<XT, 32, 4, RED, IT>(p, s);
    }
}

template <typename IT, typename XT>
static tiga_status launch_bwd_g(const CsrParams& p, int G, int VPL, cudaStream_t s) {
#define TIGA_BWD(GG, VV) csr_backward_sum_kernel<GG, VV, IT, XT><<<counted((unsigned)p.ntiles), CSR_THREADS, 0, s>>>(p); break
    switch (G) {
        case 1: TIGA_BWD(1, 1);
        case 2: TIGA_BWD(2, 1);
        case 4: TIGA_BWD(4, 1);
        case 8: TIGA_BWD(8, 1);
        case 16: TIGA_BWD(16, 1);
        default:
            if (VPL == 1) { TIGA_BWD(32, 1); }
            if (VPL == 2) { TIGA_BWD(32, 2); }
            TIGA_BWD(32, 4);
    }
#undef TIGA_BWD
    return launch_status();
}

// entries of the per-tile / per-chunk workspace arrays: tiles of the tile kernels, or chunks of the row-class path
// (at most E / chunk full chunks plus one partial chunk per chunked row, and a chunked row has more than a chunk)
static size_t work_slots(const tiga_csr* g, bool narrow_rows) {
    const size_t tiles = (size_t)num_tiles(g) + 1, chunks = (size_t)(2 * g->n_edges / row_huge_of(g)) + 2;
    return (narrow_rows && chunks > tiles) ? chunks : tiles;
}

static tiga_status check_csr(const tiga_csr* g) {
    if (!g) return TIGA_ERR_INVALID_ARG;
    if (g->n_dst < 0 || g->n_src < 0 || g->n_edges < 0) return TIGA_ERR_INVALID_ARG;
    if (g->rowptr_type != TIGA_I32 && g->rowptr_type != TIGA_I64) return TIGA_ERR_INVALID_ARG;
    if (!g->rowptr || !aligned16(g->rowptr)) return TIGA_ERR_INVALID_ARG;
    if (g->n_edges > 0 && (!g->col || !aligned16(g->col))) return TIGA_ERR_INVALID_ARG;
    if (g->rowptr_type == TIGA_I32 && g->n_edges > 0x7fffffffLL) return TIGA_ERR_INVALID_ARG;
    if (g->n_dst > 0x7fffffffLL || g->n_src > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    if (num_tiles(g) > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    return TIGA_OK;
}

static tiga_status check_features(int32_t F, tiga_dtype dt, int* nvec, int* G, int* VPL) {
    if (F <= 0) return TIGA_ERR_INVALID_ARG;
    if (dt != TIGA_F32 && dt != TIGA_F16) return TIGA_ERR_INVALID_ARG;
    const int vw = dt == TIGA_F32 ? 4 : 8;
    if (F % vw) return TIGA_ERR_UNSUPPORTED;
    *nvec = F / vw;
    return pick_shape(*nvec, G, VPL) ? TIGA_OK : TIGA_ERR_UNSUPPORTED;
}

static bool known_reducer(tiga_reducer r) { return r == TIGA_SUM || r == TIGA_MAX || r == TIGA_MAX64; }
static bool is_max(tiga_reducer r) { return r == TIGA_MAX || r == TIGA_MAX64; }
static size_t arg_bytes(tiga_reducer r) { return r == TIGA_MAX64 ? sizeof(int64_t) : sizeof(int32_t); }
// workspace array of edge positions, typed by the reducer
static void* take_args(Carver& cv, tiga_reducer r, size_t n) {
    if (!is_max(r)) return nullptr;
    return r == TIGA_MAX64 ? static_cast<void*>(cv.take<int64_t>(n)) : static_cast<void*>(cv.take<int32_t>(n));
}

}  // namespace tiga

using namespace tiga;

extern "C" size_t tiga_csr_workspace_bytes(const tiga_csr* g, int32_t F, tiga_dtype x_dtype, tiga_reducer reducer, int backward) {
    if (!g || F <= 0 || g->n_dst < 0 || g->n_edges < 0) return 0;
    if (backward) return 256;
    const size_t nt = work_slots(g, (size_t)F * (x_dtype == TIGA_F16 ? 2 : 4) <= 32);      // feature rows of at most 32 bytes: row-class path
    size_t b = align_up(nt * sizeof(int32_t), 256) + align_up(nt * F * sizeof(float), 256);
    if (is_max(reducer)) b += align_up(nt * F * arg_bytes(reducer), 256);
    b += 256 + align_up(nt * sizeof(int4), 256);      // queue of huge-row chunks (narrow-row path)
    return b + 256;
}

extern "C" tiga_status tiga_validate_csr(const tiga_csr* g, int level, void* ws, size_t ws_bytes, void* stream) {
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    if (level == 0) return TIGA_OK;
    if (!ws || ws_bytes < 16) return TIGA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int* flags = static_cast<int*>(ws);
    TIGA_CUDA_TRY(cudaMemsetAsync(flags, 0, sizeof(int), s));
    const long long work = g->n_dst > g->n_edges ? g->n_dst : g->n_edges;
    long long blocks = (work + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    if (g->rowptr_type == TIGA_I32)
        validate_kernel<int32_t><<<counted((unsigned)blocks), 256, 0, s>>>(static_cast<const int32_t*>(g->rowptr), g->col, g->n_dst, g->n_src, g->n_edges, flags);
    else
        validate_kernel<int64_t><<<counted((unsigned)blocks), 256, 0, s>>>(static_cast<const int64_t*>(g->rowptr), g->col, g->n_dst, g->n_src, g->n_edges, flags);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;
    int h = 0;
    TIGA_CUDA_TRY(cudaMemcpyAsync(&h, flags, sizeof(int), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));
    return h ? TIGA_ERR_INVALID_GRAPH : TIGA_OK;
}

extern "C" tiga_status tiga_apply_csr(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                                      const float* w, const tiga_msg* msg, tiga_reducer reducer,
                                      float* out, void* argmax, void* ws, size_t ws_bytes, void* stream) {
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    int nvec, G, VPL;
    st = check_features(F, x_dtype, &nvec, &G, &VPL);
    if (st != TIGA_OK) return st;
    if (!known_reducer(reducer)) return TIGA_ERR_INVALID_ARG;
    if (!msg) return TIGA_ERR_INVALID_ARG;
    if (msg->kind == TIGA_MSG_COPY) { if (w) return TIGA_ERR_INVALID_ARG; }
    else if (msg->kind == TIGA_MSG_WEIGHTED) { if (!w && g->n_edges > 0) return TIGA_ERR_INVALID_ARG; }
    else return TIGA_ERR_UNSUPPORTED;
    if (g->n_dst == 0) return TIGA_OK;
    if (!out || !aligned16(out) || (g->n_src > 0 && (!x || !aligned16(x)))) return TIGA_ERR_INVALID_ARG;
    if (w && !aligned16(w)) return TIGA_ERR_INVALID_ARG;
    if (is_max(reducer)) {
        if (!argmax || !aligned16(argmax)) return TIGA_ERR_INVALID_ARG;
        if (reducer == TIGA_MAX && g->n_edges > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;     // 32-bit positions: use TIGA_MAX64
    }
    if (!ws || !aligned16(ws) || ws_bytes < tiga_csr_workspace_bytes(g, F, x_dtype, reducer, 0)) return TIGA_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CsrParams p{};
    p.rowptr = g->rowptr; p.col = g->col; p.w = w; p.x = x; p.out = out; p.arg = argmax;
    p.n_dst = g->n_dst; p.n_edges = g->n_edges; p.n_src = g->n_src; p.F = F; p.nvec = nvec;
    p.ntiles = num_tiles(g);
    Carver cv(ws);
    const size_t slots = work_slots(g, nvec <= 2);
    p.carry_row = cv.take<int32_t>(slots);
    p.carry_val = cv.take<float>(slots * F);
    p.carry_arg = take_args(cv, reducer, slots * F);
    p.huge_count = cv.take<int>(1);
    p.huge_list = cv.take<int4>(slots);
    p.row_huge = row_huge_of(g);
    p.ntiles = num_tiles(g, reducer == TIGA_SUM ? CSR_TILE : CSR_TILE_MAX);      // the launch's tiles (the arrays hold at least as many)

    const bool i64 = g->rowptr_type == TIGA_I64;
    if (reducer == TIGA_MAX64) {
        // 64-bit positions only make sense with 64-bit row offsets; a 32-bit rowptr still works
        if (x_dtype == TIGA_F32) st = i64 ? launch_fwd_g<float, 2, int64_t>(p, G, VPL, s) : launch_fwd_g<float, 2, int32_t>(p, G, VPL, s);
        else st = i64 ? launch_fwd_g<__half, 2, int64_t>(p, G, VPL, s) : launch_fwd_g<__half, 2, int32_t>(p, G, VPL, s);
    } else if (x_dtype == TIGA_F32) {
        if (reducer == TIGA_SUM) st = i64 ? launch_fwd_g<float, 0, int64_t>(p, G, VPL, s) : launch_fwd_g<float, 0, int32_t>(p, G, VPL, s);
        else st = i64 ? launch_fwd_g<float, 1, int64_t>(p, G, VPL, s) : launch_fwd_g<float, 1, int32_t>(p, G, VPL, s);
    } else {
        if (reducer == TIGA_SUM) st = i64 ? launch_fwd_g<__half, 0, int64_t>(p, G, VPL, s) : launch_fwd_g<__half, 0, int32_t>(p, G, VPL, s);
        else st = i64 ? launch_fwd_g<__half, 1, int64_t>(p, G, VPL, s) : launch_fwd_g<__half, 1, int32_t>(p, G, VPL, s);
    }
    if (st != TIGA_OK) return st;
    if (nvec <= 2) return TIGA_OK;             // the row-class path has no tile carry-outs
    const long long work = p.ntiles * F;
    const unsigned fix_blocks = (unsigned)((work + 255) / 256);
    if (reducer == TIGA_SUM) csr_fixup_kernel<0><<<counted(fix_blocks), 256, 0, s>>>(p);
    else if (reducer == TIGA_MAX) csr_fixup_kernel<1><<<counted(fix_blocks), 256, 0, s>>>(p);
    else csr_fixup_kernel<2><<<counted(fix_blocks), 256, 0, s>>>(p);
    return launch_status();
}

// ---- built-in scratch for callers that cannot allocate -------------------------------------
// The array is part of this library's device image, so every GPU that loads the library
// carries it until the process exits.  In host code its name is only a handle for the
// runtime: the address a kernel can use comes from cudaGetSymbolAddress, looked up once per
// device with that device current.
static __device__ __align__(256) unsigned char g_builtin_ws[TIGA_BUILTIN_WS_BYTES];

static tiga_status builtin_ws_address(void** out) {
    constexpr int MAX_DEVICES = 64;
    static void* cached[MAX_DEVICES] = {};
    static std::mutex lock;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return TIGA_ERR_CUDA;
    std::lock_guard<std::mutex> guard(lock);
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_builtin_ws) != cudaSuccess || !ptr) return TIGA_ERR_CUDA;
        cached[dev] = ptr;
    }
    *out = cached[dev];
    return TIGA_OK;
}

extern "C" tiga_status tiga_apply_csr_builtin_ws(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                                                 const float* w, const tiga_msg* msg, tiga_reducer reducer,
                                                 float* out, void* argmax, void* stream) {
    // capacity first: a refusal touches neither the device nor the array
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    if (F <= 0) return TIGA_ERR_INVALID_ARG;
    if (!known_reducer(reducer)) return TIGA_ERR_INVALID_ARG;
    if (tiga_csr_workspace_bytes(g, F, x_dtype, reducer, 0) > (size_t)TIGA_BUILTIN_WS_BYTES) return TIGA_ERR_TOO_LARGE;
    void* ws = nullptr;
    st = builtin_ws_address(&ws);
    if (st != TIGA_OK) return st;
    return tiga_apply_csr(g, x, x_dtype, F, w, msg, reducer, out, argmax, ws, (size_t)TIGA_BUILTIN_WS_BYTES, stream);
}

// ---- planned forward (hot-source plan; see csr_plan.cu) ------------------------------------
extern "C" size_t tiga_csr_planned_workspace_bytes(const tiga_csr* g, const tiga_csr_plan* plan, int32_t F, tiga_dtype x_dtype,
                                                   tiga_reducer reducer) {
    if (!g || !plan || F <= 0) return 0;
    const size_t row_bytes = (size_t)F * (x_dtype == TIGA_F32 ? 4 : 2);
    return align_up((size_t)plan->n_hot * row_bytes + 256, 256) + tiga_csr_workspace_bytes(g, F, x_dtype, reducer, 0);
}

extern "C" tiga_status tiga_apply_csr_planned(const tiga_csr* g, const tiga_csr_plan* plan, const void* plan_buf,
                                              const void* x, tiga_dtype x_dtype, int32_t F, const float* w, const tiga_msg* msg,
                                              tiga_reducer reducer, float* out, void* argmax,
                                              void* ws, size_t ws_bytes, void* stream) {
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    if (!plan || !plan_buf || !aligned16(plan_buf)) return TIGA_ERR_INVALID_ARG;
    if (plan->n_dst != g->n_dst || plan->n_src != g->n_src || plan->n_edges != g->n_edges) return TIGA_ERR_INVALID_ARG;
    int nvec, G, VPL;
    st = check_features(F, x_dtype, &nvec, &G, &VPL);
    if (st != TIGA_OK) return st;
    if (nvec > 2) return TIGA_ERR_UNSUPPORTED;            // feature rows of at most 32 bytes: the case the plan exists for
    if (!known_reducer(reducer)) return TIGA_ERR_INVALID_ARG;
    if (reducer == TIGA_MAX && g->n_edges > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    if (!msg) return TIGA_ERR_INVALID_ARG;
    if (msg->kind == TIGA_MSG_COPY) { if (w) return TIGA_ERR_INVALID_ARG; }
    else if (msg->kind == TIGA_MSG_WEIGHTED) { if (!w) return TIGA_ERR_INVALID_ARG; }
    else return TIGA_ERR_UNSUPPORTED;
    if (g->n_dst == 0) return TIGA_OK;
    if (!out || !aligned16(out) || !x || !aligned16(x) || (w && !aligned16(w))) return TIGA_ERR_INVALID_ARG;
    if (is_max(reducer) && (!argmax || !aligned16(argmax))) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_csr_planned_workspace_bytes(g, plan, F, x_dtype, reducer)) return TIGA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const char* base = static_cast<const char*>(plan_buf);

    CsrParams p{};
    p.rowptr = g->rowptr; p.col = reinterpret_cast<const int32_t*>(base + plan->off_col);
    p.w = w; p.x = x; p.out = out; p.arg = argmax;
    p.n_dst = g->n_dst; p.n_edges = g->n_edges; p.n_src = g->n_src; p.F = F; p.nvec = nvec;
    p.ntiles = num_tiles(g);
    Carver cv(ws);
    const size_t row_bytes = (size_t)F * (x_dtype == TIGA_F32 ? 4 : 2);
    void* hot = cv.take<unsigned char>((size_t)plan->n_hot * row_bytes + 256);
    p.x_hot = hot; p.n_hot = (int)plan->n_hot;
    p.n_src = g->n_src + plan->n_hot;                      // range of the rewritten indices
    const size_t slots = work_slots(g, nvec <= 2);
    p.carry_row = cv.take<int32_t>(slots);
    p.carry_val = cv.take<float>(slots * F);
    p.carry_arg = take_args(cv, reducer, slots * F);
    p.huge_count = cv.take<int>(1);
    p.huge_list = cv.take<int4>(slots);
    p.row_huge = row_huge_of(g);
    st = launch_gather_hot(x, reinterpret_cast<const int32_t*>(base + plan->off_hot_id), plan->n_hot, nvec, hot, s);
    if (st != TIGA_OK) return st;
    const bool i64 = g->rowptr_type == TIGA_I64;
    if (reducer == TIGA_MAX64) {
        if (x_dtype == TIGA_F32) return i64 ? launch_fwd_narrow<float, 2, int64_t, true>(p, s) : launch_fwd_narrow<float, 2, int32_t, true>(p, s);
        return i64 ? launch_fwd_narrow<__half, 2, int64_t, true>(p, s) : launch_fwd_narrow<__half, 2, int32_t, true>(p, s);
    }
    if (x_dtype == TIGA_F32) {
        if (reducer == TIGA_SUM) return i64 ? launch_fwd_narrow<float, 0, int64_t, true>(p, s) : launch_fwd_narrow<float, 0, int32_t, true>(p, s);
        return i64 ? launch_fwd_narrow<float, 1, int64_t, true>(p, s) : launch_fwd_narrow<float, 1, int32_t, true>(p, s);
    }
    if (reducer == TIGA_SUM) return i64 ? launch_fwd_narrow<__half, 0, int64_t, true>(p, s) : launch_fwd_narrow<__half, 0, int32_t, true>(p, s);
    return i64 ? launch_fwd_narrow<__half, 1, int64_t, true>(p, s) : launch_fwd_narrow<__half, 1, int32_t, true>(p, s);
}

extern "C" tiga_status tiga_apply_csr_backward(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                                               const float* w, const tiga_msg* msg, tiga_reducer reducer,
                                               const float* grad_out, const void* argmax,
                                               float* grad_x, float* grad_w,
                                               void* ws, size_t ws_bytes, void* stream) {
    (void)ws; (void)ws_bytes;
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    int nvec, G, VPL;
    st = check_features(F, x_dtype, &nvec, &G, &VPL);        // the feature rows must be whole 16-byte vectors
    if (st != TIGA_OK) return st;
    st = check_features(F, TIGA_F32, &nvec, &G, &VPL);       // lanes own four fp32 gradient values whatever x's type
    if (st != TIGA_OK) return st;
    if (!known_reducer(reducer)) return TIGA_ERR_INVALID_ARG;
    if (!msg) return TIGA_ERR_INVALID_ARG;
    if (msg->kind == TIGA_MSG_COPY) { if (w) return TIGA_ERR_INVALID_ARG; }
    else if (msg->kind == TIGA_MSG_WEIGHTED) { if (!w && g->n_edges > 0) return TIGA_ERR_INVALID_ARG; }
    else return TIGA_ERR_UNSUPPORTED;
    if (g->n_dst > 0 && (!grad_out || !aligned16(grad_out))) return TIGA_ERR_INVALID_ARG;
    if (g->n_src > 0 && (!x || !aligned16(x))) return TIGA_ERR_INVALID_ARG;
    if ((grad_x && !aligned16(grad_x)) || (grad_w && !aligned16(grad_w)) || (w && !aligned16(w))) return TIGA_ERR_INVALID_ARG;
    if (is_max(reducer)) {
        if (g->n_dst > 0 && (!argmax || !aligned16(argmax))) return TIGA_ERR_INVALID_ARG;
        if (reducer == TIGA_MAX && g->n_edges > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (grad_x && g->n_src > 0) TIGA_CUDA_TRY(cudaMemsetAsync(grad_x, 0, (size_t)g->n_src * F * sizeof(float), s));
    if (is_max(reducer) && grad_w && g->n_edges > 0) TIGA_CUDA_TRY(cudaMemsetAsync(grad_w, 0, (size_t)g->n_edges * sizeof(float), s));
    if (g->n_dst == 0 || g->n_edges == 0 || (!grad_x && !grad_w)) return TIGA_OK;

    CsrParams p{};
    p.rowptr = g->rowptr; p.col = g->col; p.w = w; p.x = x; p.arg = const_cast<void*>(argmax);
    p.n_dst = g->n_dst; p.n_edges = g->n_edges; p.n_src = g->n_src; p.F = F; p.nvec = nvec;
    p.ntiles = num_tiles(g, CSR_TILE_BWD);
    p.gy = grad_out; p.gx = grad_x; p.gw = grad_w;
    if (reducer == TIGA_SUM) {
        if (x_dtype == TIGA_F16)
            return g->rowptr_type == TIGA_I64 ? launch_bwd_g<int64_t, __half>(p, G, VPL, s) : launch_bwd_g<int32_t, __half>(p, G, VPL, s);
        return g->rowptr_type == TIGA_I64 ? launch_bwd_g<int64_t, float>(p, G, VPL, s) : launch_bwd_g<int32_t, float>(p, G, VPL, s);
    }
    // Measured on R-MAT relations with F = 64: the four-features-per-thread form wins once the gradient table
    // no longer fits L2 (scale 20, 268 MB: 0.47 against 0.49 ms), the thread-per-feature form below that
    // (scale 18, 67 MB: 0.13 against 0.16 ms).
    const bool grouped = (size_t)g->n_src * F * sizeof(float) > ((size_t)128 << 20);
    const unsigned blocks = (unsigned)(((grouped ? g->n_dst * F / 4 : g->n_dst * F) + 255) / 256);
#define TIGA_MAX_BWD(XT, RR)                                                                   \
    do {                                                                                       \
        if (grouped) csr_backward_max_kernel<XT, RR><<<counted(blocks), 256, 0, s>>>(p);       \
        else csr_backward_max_each_kernel<XT, RR><<<counted(blocks), 256, 0, s>>>(p);          \
    } while (0)
    if (reducer == TIGA_MAX) {
        if (x_dtype == TIGA_F16) TIGA_MAX_BWD(__half, 1); else TIGA_MAX_BWD(float, 1);
    } else {
        if (x_dtype == TIGA_F16) TIGA_MAX_BWD(__half, 2); else TIGA_MAX_BWD(float, 2);
    }
#undef TIGA_MAX_BWD
    return launch_status();
}

extern "C" tiga_status tiga_csr_degree_histogram(const tiga_csr* g, int64_t* hist, int64_t nbins,
                                                 int64_t* max_degree, void* stream) {
    tiga_status st = check_csr(g);
    if (st != TIGA_OK) return st;
    if (!hist || !max_degree || nbins < 1 || nbins > 8192) return TIGA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TIGA_CUDA_TRY(cudaMemsetAsync(hist, 0, (size_t)nbins * sizeof(int64_t), s));
    TIGA_CUDA_TRY(cudaMemsetAsync(max_degree, 0, sizeof(int64_t), s));
    if (g->n_dst == 0) return TIGA_OK;
    // one CTA of 1024 threads per SM (eight row-offset loads in flight per thread): every CTA ends with one global atomic per non-empty bin, so few
    // large CTAs keep that flush (CTAs x bins atomics on nbins addresses) short
    long long blocks = (g->n_dst + 4095) / 4096;
    if (blocks > 148) blocks = 148;
    const size_t sm = (size_t)nbins * sizeof(unsigned int);
    if (g->rowptr_type == TIGA_I32)
        degree_hist_kernel<int32_t><<<counted((unsigned)blocks), 1024, sm, s>>>(static_cast<const int32_t*>(g->rowptr), g->n_dst, (int)nbins,
                                                                   reinterpret_cast<unsigned long long*>(hist), reinterpret_cast<unsigned long long*>(max_degree));
    else
        degree_hist_kernel<int64_t><<<counted((unsigned)blocks), 1024, sm, s>>>(static_cast<const int64_t*>(g->rowptr), g->n_dst, (int)nbins,
                                                                   reinterpret_cast<unsigned long long*>(hist), reinterpret_cast<unsigned long long*>(max_degree));
    return launch_status();
}

extern "C" int64_t tiga_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

extern "C" uint32_t tiga_checked_status(int reset) {
#ifdef TIGA_CHECKED
    if (cudaDeviceSynchronize() != cudaSuccess) return 0x80000000u;
    const bool r = reset != 0;
    return check_status_csr(r) | check_status_csr_plan(r) | check_status_csr_attention(r) | check_status_radius(r) |
           check_status_radius_lj(r) | check_status_radius_mlp(r) | check_status_knn(r);
#else
    (void)reset;
    return 0u;
#endif
}

extern "C" int tiga_is_checked_build(void) {
#ifdef TIGA_CHECKED
    return 1;
#else
    return 0;
#endif
}

extern "C" const char* tiga_status_string(tiga_status s) {
    switch (s) {
        case TIGA_OK: return "ok";
        case TIGA_ERR_INVALID_ARG: return "invalid argument";
        case TIGA_ERR_UNSUPPORTED: return "unsupported combination";
        case TIGA_ERR_WORKSPACE: return "workspace missing or too small";
        case TIGA_ERR_CUDA: return "CUDA runtime error";
        case TIGA_ERR_INVALID_GRAPH: return "malformed CSR relation";
        case TIGA_ERR_TOO_LARGE: return "problem exceeds the library's built-in scratch capacity";
        case TIGA_ERR_INVALID_POINTS: return "a point coordinate is not finite or lies outside the box";
    }
    return "unknown status";
}

namespace tiga { unsigned check_status_csr(bool reset) { return read_check_status(reset); } }
