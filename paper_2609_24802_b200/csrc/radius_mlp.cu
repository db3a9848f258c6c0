// Edge neural network over the generated radius relation (paper Appendix A):
//     y_i = sum over j in N(i) of [ W2 ReLU( W1 [p_j - p_i ; x_j] + b1 ) + b2 ]
// fused with the cell-directory traversal, and its reverse mode with the membership frozen
// (Section 5), which recomputes the activations per pair instead of storing them and gives
// gradients with respect to node features, positions and the four parameter arrays.
//
// Same skeleton as the other radius traversals: one warp per query cell (here in a persistent
// loop over cells), the 27-cell stencil staged in shared memory in cell-local coordinates,
// one staged candidate per lane tested against eight queries, ballot compaction into one list
// per query.  What differs is phase B: every lane takes one accepted pair and evaluates the
// whole network for it with the weights broadcast from shared memory (input padded to 4 KQ,
// hidden width HID in registers).  The pairs of all queries of a batch form one flat sequence,
// 32 per step, so short neighbour lists do not leave lanes idle; per-query sums are segmented
// shuffle reductions (fixed order: reproducible).
//
// Backward, owner computes: for query k and neighbour m a lane evaluates the pair twice,
//   (k <- m) gives the parameter gradients and -ubar[0:3] for pbar_k,
//   (m <- k) gives xbar_k and +ubar[0:3] for pbar_k,
// so feature and position gradients need no atomics.  Parameter gradients: the 32 pairs of a
// step park (hbar, u, a, ybar) in shared memory, then every lane accumulates "its" parameter
// entries over those pairs in registers; at the end warps fold into the CTA's shared copy and
// the CTA adds that to global memory with one atomic per entry.
#include "radius_shared.cuh"
#include <type_traits>

namespace tiga {

constexpr int MLP_STAGE_CAP = 256;
constexpr int MLP_QCAP = 80;
constexpr int MLP_QSTRIDE = MLP_QCAP + 1;
constexpr int MLP_DIN = 16;             // padded input width (3 + f_in <= 16)

template <int HID, bool BWD> struct MlpSmem {
    static constexpr int W_FLOATS = HID * MLP_DIN + HID + 4 * HID + 4;          // W1 (padded), b1, W2 (4 rows), b2
    static constexpr int CTA_BYTES = (W_FLOATS * (BWD ? 2 : 1) * 4 + 15) / 16 * 16;   // weights (+ gradient accumulators)
    static constexpr int STAGE_BYTES = (MLP_STAGE_CAP + STAGE_PAD) * 16;
    static constexpr int LIST_BYTES = (QB * MLP_QSTRIDE * 4 + 15) / 16 * 16;
    static constexpr int ACC_W = 16;                                             // per-query accumulator: outputs, or pbar (3) + xbar (13)
    static constexpr int MISC_BYTES = QB * 16 + QB * 4 * 2 + QB * ACC_W * 4;
    static constexpr int PAIR_STRIDE = 2 * HID + MLP_DIN + 4 + 1;                // hbar, u, a, ybar (+1: odd stride)
    static constexpr int PAIR_BYTES = BWD ? (32 * PAIR_STRIDE * 4 + 15) / 16 * 16 : 0;
    static constexpr int PER_WARP = STAGE_BYTES + LIST_BYTES + MISC_BYTES + PAIR_BYTES;
    static_assert(PER_WARP % 16 == 0, "the stage and the queries are accessed as 16-byte vectors");
    static constexpr int TOTAL = CTA_BYTES + TRAV_WARPS * PER_WARP;
};

template <int HID, int KQ>
__device__ __forceinline__ void mlp_forward(const float* sW1, const float* sb1, const float* sW2, const float* sb2,
                                            const float (&u)[4 * KQ], float (&h)[HID], float (&m)[4]) {
#pragma unroll
    for (int a = 0; a < HID; ++a) {
        float s = sb1[a];
        const float4* w = reinterpret_cast<const float4*>(sW1 + a * MLP_DIN);
#pragma unroll
        for (int q = 0; q < KQ; ++q) {
            const float4 w4 = w[q];
            s = fmaf(w4.x, u[4 * q], s); s = fmaf(w4.y, u[4 * q + 1], s);
            s = fmaf(w4.z, u[4 * q + 2], s); s = fmaf(w4.w, u[4 * q + 3], s);
        }
        h[a] = s;
    }
#pragma unroll
    for (int o = 0; o < 4; ++o) {
        float s = sb2[o];
#pragma unroll
        for (int a = 0; a < HID; ++a) s = fmaf(sW2[o * HID + a], fmaxf(h[a], 0.f), s);
        m[o] = s;
    }
}

// hbar = (W2^T ybar) * [h > 0],  ubar = W1^T hbar.  hbar is consumed entry by entry (and parked in
// shared memory where the parameter gradients need it), so it never occupies HID registers.
template <int HID, int KQ, bool STORE>
__device__ __forceinline__ void mlp_backward(const float* sW1, const float* sW2, const float (&h)[HID], const float (&gy)[4],
                                             float* hb_out, float (&ub)[4 * KQ]) {
#pragma unroll
    for (int c = 0; c < 4 * KQ; ++c) ub[c] = 0.f;
#pragma unroll
    for (int a = 0; a < HID; ++a) {
        float s = sW2[a] * gy[0];
        s = fmaf(sW2[HID + a], gy[1], s); s = fmaf(sW2[2 * HID + a], gy[2], s); s = fmaf(sW2[3 * HID + a], gy[3], s);
        const float hb = h[a] > 0.f ? s : 0.f;
        if (STORE) hb_out[a] = hb;
        const float4* w = reinterpret_cast<const float4*>(sW1 + a * MLP_DIN);
#pragma unroll
        for (int q = 0; q < KQ; ++q) {
            const float4 w4 = w[q];
            ub[4 * q] = fmaf(w4.x, hb, ub[4 * q]); ub[4 * q + 1] = fmaf(w4.y, hb, ub[4 * q + 1]);
            ub[4 * q + 2] = fmaf(w4.z, hb, ub[4 * q + 2]); ub[4 * q + 3] = fmaf(w4.w, hb, ub[4 * q + 3]);
        }
    }
}

// resident CTAs per SM the kernel is compiled for (register budget) and launched with (persistent grid)
template <int HID, bool BWD> constexpr int mlp_ctas_per_sm() { return BWD ? (HID <= 16 ? 3 : 2) : (HID <= 16 ? 4 : 3); }

template <int HID, int KQ, bool BWD, bool MI>
__global__ void __launch_bounds__(TRAV_THREADS, mlp_ctas_per_sm<HID, BWD>()) radius_mlp_kernel(const __grid_constant__ RadiusParams p) {
    using SM = MlpSmem<HID, BWD>;
    constexpr unsigned FULL = 0xffffffffu;
    constexpr int KU = 4 * KQ;
    constexpr int PS = SM::PAIR_STRIDE;
    extern __shared__ __align__(16) unsigned char s_raw[];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int Fin = p.Fin, Fout = p.Fout, K = 3 + p.Fin;

    // ---- CTA: weights into shared memory (zero padded), gradient accumulators cleared
    float* sW1 = reinterpret_cast<float*>(s_raw);
    float* sb1 = sW1 + HID * MLP_DIN;
    float* sW2 = sb1 + HID;
    float* sb2 = sW2 + 4 * HID;
    float* sG = sb2 + 4;                       // BWD: same layout as the weights
    for (int e = threadIdx.x; e < HID * MLP_DIN; e += TRAV_THREADS) {
        const int a = e / MLP_DIN, k = e % MLP_DIN;
        sW1[e] = k < K ? p.W1[a * K + k] : 0.f;
    }
    for (int e = threadIdx.x; e < HID; e += TRAV_THREADS) sb1[e] = p.b1[e];
    for (int e = threadIdx.x; e < 4 * HID; e += TRAV_THREADS) sW2[e] = (e / HID) < Fout ? p.W2[e] : 0.f;
    if (threadIdx.x < 4) sb2[threadIdx.x] = threadIdx.x < Fout ? p.b2[threadIdx.x] : 0.f;
    if (BWD) for (int e = threadIdx.x; e < SM::W_FLOATS; e += TRAV_THREADS) sG[e] = 0.f;
    __syncthreads();

    unsigned char* base = s_raw + SM::CTA_BYTES + (size_t)wib * SM::PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);
    int* list = reinterpret_cast<int*>(base + SM::STAGE_BYTES);
    float4* s_q = reinterpret_cast<float4*>(base + SM::STAGE_BYTES + SM::LIST_BYTES);
    int* s_n = reinterpret_cast<int*>(s_q + QB);
    int* s_tot = s_n + QB;
    float* s_acc = reinterpret_cast<float*>(s_tot + QB);          // [QB][ACC_W] sums of the drain in progress
    float* pairbuf = reinterpret_cast<float*>(base + SM::STAGE_BYTES + SM::LIST_BYTES + SM::MISC_BYTES);

    const bool mi0 = MI && p.periodic[0] && p.nc[0] == 1, mi1 = MI && p.periodic[1] && p.nc[1] == 1, mi2 = MI && p.periodic[2] && p.nc[2] == 1;
    const unsigned lt_mask = (1u << lane) - 1u;
    auto fold = [&](float& dx, float& dy, float& dz) {
        if (MI) {
            if (mi0) dx -= p.len[0] * rintf(dx * p.inv_len[0]);
            if (mi1) dy -= p.len[1] * rintf(dy * p.inv_len[1]);
            if (mi2) dz -= p.len[2] * rintf(dz * p.inv_len[2]);
        }
    };

    // parameter-gradient entries owned by this lane (BWD): W1[a0 + 2 i][k1], W2[o][lane], b1[lane], b2[lane]
    const int k1 = lane & 15, a0 = lane >> 4;
    float gW1acc[BWD ? HID / 2 : 1], gW2acc[4] = {0.f, 0.f, 0.f, 0.f}, gb1acc = 0.f, gb2acc = 0.f;
#pragma unroll
    for (int i = 0; i < (BWD ? HID / 2 : 1); ++i) gW1acc[i] = 0.f;

    // work items: every cell (of a cell with more than QDENSE points only its first QSLICE queries), then
    // the queued slices of the dense cells, so that a clustered input spreads over all warps
    const int nitems = p.ncells + *p.q_count;
    for (int item = blockIdx.x * TRAV_WARPS + wib; item < nitems; item += gridDim.x * TRAV_WARPS) {
        int cellid, qs0, qe0;
        if (item < p.ncells) {
            cellid = item;
            qs0 = p.cell_start[cellid]; qe0 = p.cell_start[cellid + 1];
            if (qe0 - qs0 > QDENSE) qe0 = qs0 + QSLICE;
        } else {
            const int2 it = p.q_items[item - p.ncells];
            cellid = it.x;
            qs0 = p.cell_start[cellid] + it.y;
            qe0 = slice_end(qs0, p.cell_start[cellid + 1]);
        }
        if (qs0 == qe0) continue;
        const int c[3] = {cellid % p.nc[0], (cellid / p.nc[0]) % p.nc[1], cellid / (p.nc[0] * p.nc[1])};
        const float org[3] = {(float)c[0] * p.hcell[0], (float)c[1] * p.hcell[1], (float)c[2] * p.hcell[2]};

        auto process_chunk = [&](const int ns, const bool first_chunk) {
            if (lane < STAGE_PAD) stage[ns + lane] = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-1));
            for (int qb0 = qs0; qb0 < qe0; qb0 += QB) {
                const int nq = (qe0 - qb0 < QB) ? qe0 - qb0 : QB;
                __syncwarp();
                if (lane < nq) {
                    const float4 pq = p.spos[qb0 + lane];
                    s_q[lane] = make_float4(pq.x - org[0], pq.y - org[1], pq.z - org[2], pq.w);
                    s_tot[lane] = 0;
                }
                __syncwarp();
                int qcnt[QB];
#pragma unroll
                for (int q = 0; q < QB; ++q) qcnt[q] = 0;
                bool first = first_chunk;

                auto drain = [&]() {
                    constexpr int ACC_W = SM::ACC_W;
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int q = 0; q < QB; ++q) { s_n[q] = qcnt[q]; s_tot[q] += qcnt[q]; }
                    }
                    for (int e = lane; e < QB * ACC_W; e += 32) s_acc[e] = 0.f;
                    __syncwarp();
                    // The accepted pairs of all queries of the batch form one flat sequence, 32 pairs per step
                    // whatever the list lengths (a query with a dozen neighbours would otherwise leave most of
                    // a step idle).  Lanes of one query are neighbours in that sequence, so per-query sums are
                    // segmented reductions; the first lane of a segment adds the sum to the query's accumulator.
                    int pre[QB + 1];
                    pre[0] = 0;
#pragma unroll
                    for (int q = 0; q < QB; ++q) pre[q + 1] = pre[q] + (q < nq ? s_n[q] : 0);
                    const int npairs = pre[QB];
                    for (int t0 = 0; t0 < npairs; t0 += 32) {
                        const int f = t0 + lane;
                        const bool valid = f < npairs;
                        int q = 0;
#pragma unroll
                        for (int j = 1; j < QB; ++j) q += (f >= pre[j]) ? 1 : 0;
                        q = q < nq ? q : nq - 1;
                        int tq = 0;
#pragma unroll
                        for (int j = 0; j < QB; ++j) tq = (j == q) ? f - pre[j] : tq;
                        const int key = valid ? q : -1 - lane;               // idle lanes form segments of their own
                        const float4 qv = s_q[q];
                        const int oq = checked(__float_as_int(qv.w), p.n, CHECK_POINT);
                        float4 pj = make_float4(0.f, 0.f, 0.f, __int_as_float(0));
                        if (valid) pj = stage[list[q * MLP_QSTRIDE + tq]];
                        float dx = pj.x - qv.x, dy = pj.y - qv.y, dz = pj.z - qv.z;      // source minus destination
                        fold(dx, dy, dz);
                        constexpr int NV = BWD ? KU : 4;
                        float red[NV];
#pragma unroll
                        for (int i = 0; i < NV; ++i) red[i] = 0.f;
                        if constexpr (!BWD) {
                            if (valid) {
                                float u[KU], h[HID], m[4];
                                u[0] = dx; u[1] = dy; u[2] = dz;
                                const float* xr = p.feat + (size_t)checked(__float_as_int(pj.w), p.n, CHECK_POINT) * Fin;
#pragma unroll
                                for (int k = 3; k < KU; ++k) u[k] = (k - 3 < Fin) ? __ldg(xr + k - 3) : 0.f;
                                mlp_forward<HID, KQ>(sW1, sb1, sW2, sb2, u, h, m);
#pragma unroll
                                for (int o = 0; o < 4; ++o) red[o] = m[o];
                            }
                        } else {
                            float* mine = pairbuf + lane * PS;
                            if (valid) {
                                const int om = checked(__float_as_int(pj.w), p.n, CHECK_POINT);
                                float gyk[4], gym[4];
#pragma unroll
                                for (int o = 0; o < 4; ++o) {
                                    gyk[o] = o < Fout ? __ldg(p.gy + (size_t)oq * Fout + o) : 0.f;
                                    gym[o] = o < Fout ? __ldg(p.gy + (size_t)om * Fout + o) : 0.f;
                                }
                                float u[KU], h[HID], m[4], ub[KU];
                                // pair (k <- m): parameter gradients and the destination part of pbar_k
                                u[0] = dx; u[1] = dy; u[2] = dz;
                                const float* xr = p.feat + (size_t)om * Fin;
#pragma unroll
                                for (int k = 3; k < KU; ++k) u[k] = (k - 3 < Fin) ? __ldg(xr + k - 3) : 0.f;
                                mlp_forward<HID, KQ>(sW1, sb1, sW2, sb2, u, h, m);
                                mlp_backward<HID, KQ, true>(sW1, sW2, h, gyk, mine, ub);       // hbar goes straight to the pair buffer
                                red[0] = -ub[0]; red[1] = -ub[1]; red[2] = -ub[2];
#pragma unroll
                                for (int a = 0; a < HID; ++a) mine[HID + MLP_DIN + a] = fmaxf(h[a], 0.f);
#pragma unroll
                                for (int k = 0; k < MLP_DIN; ++k) mine[HID + k] = k < KU ? u[k < KU ? k : 0] : 0.f;
#pragma unroll
                                for (int o = 0; o < 4; ++o) mine[2 * HID + MLP_DIN + o] = gyk[o];
                                // pair (m <- k): xbar_k and the source part of pbar_k
                                const float* xq = p.feat + (size_t)oq * Fin;
                                u[0] = -dx; u[1] = -dy; u[2] = -dz;
#pragma unroll
                                for (int k = 3; k < KU; ++k) u[k] = (k - 3 < Fin) ? __ldg(xq + k - 3) : 0.f;
                                mlp_forward<HID, KQ>(sW1, sb1, sW2, sb2, u, h, m);
                                mlp_backward<HID, KQ, false>(sW1, sW2, h, gym, nullptr, ub);
                                red[0] += ub[0]; red[1] += ub[1]; red[2] += ub[2];
#pragma unroll
                                for (int k = 3; k < KU; ++k) red[k] = ub[k];
                            }
                            __syncwarp();
                            const int np = npairs - t0 < 32 ? npairs - t0 : 32;
                            for (int pp = 0; pp < np; ++pp) {
                                const float* pb = pairbuf + pp * PS;
                                const float uk = pb[HID + k1];
#pragma unroll
                                for (int i = 0; i < HID / 2; ++i) gW1acc[i] = fmaf(pb[a0 + 2 * i], uk, gW1acc[i]);
                                if (lane < HID) {
                                    const float act = pb[HID + MLP_DIN + lane];
#pragma unroll
                                    for (int o = 0; o < 4; ++o) gW2acc[o] = fmaf(pb[2 * HID + MLP_DIN + o], act, gW2acc[o]);
                                    gb1acc += pb[lane];
                                }
                                if (lane < 4) gb2acc += pb[2 * HID + MLP_DIN + lane];
                            }
                        }
                        // segmented sums over the lanes of one query
#pragma unroll
                        for (int d = 1; d < 32; d <<= 1) {
                            const int kd = __shfl_down_sync(FULL, key, d);
                            const bool same = lane + d < 32 && kd == key;
#pragma unroll
                            for (int i = 0; i < NV; ++i) {
                                const float vd = __shfl_down_sync(FULL, red[i], d);
                                if (same) red[i] += vd;
                            }
                        }
                        const int kprev = __shfl_up_sync(FULL, key, 1);
                        if (valid && (lane == 0 || kprev != key)) {
#pragma unroll
                            for (int i = 0; i < NV; ++i) s_acc[q * ACC_W + i] += red[i];     // one first lane per query and step
                        }
                        __syncwarp();
                    }
                    // the batch's rows
                    if constexpr (!BWD) {
                        const int q = lane >> 2, o = lane & 3;
                        if (q < nq && o < Fout) {
                            float* dst = p.out + (size_t)__float_as_int(s_q[q].w) * Fout + o;
                            const float v = s_acc[q * ACC_W + o];
                            *dst = first ? v : *dst + v;
                        }
                    } else {
                        for (int e = lane; e < nq * ACC_W; e += 32) {
                            const int q = e / ACC_W, cidx = e % ACC_W;
                            const int oq = __float_as_int(s_q[q].w);
                            const float v = s_acc[e];
                            if (cidx < 3) {
                                if (p.gpos) { float* o = p.gpos + 3 * (size_t)oq + cidx; *o = first ? v : *o + v; }
                            } else if (cidx - 3 < Fin && cidx < KU) {
                                if (p.gfeat) { float* o = p.gfeat + (size_t)oq * Fin + cidx - 3; *o = first ? v : *o + v; }
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < QB; ++q) qcnt[q] = 0;
                    first = false;
                    __syncwarp();
                };

                auto phase_a = [&](const int cbase) -> bool {
                    const float4 pj = stage[cbase + lane];
                    const int idj = __float_as_int(pj.w);
                    float d2q[QB];
                    float nearest = FAR_AWAY;
#pragma unroll
                    for (int q = 0; q < QB; ++q) {
                        if (q >= nq) break;
                        const float4 qv = s_q[q];
                        float dx = qv.x - pj.x, dy = qv.y - pj.y, dz = qv.z - pj.z;
                        fold(dx, dy, dz);
                        float d2 = fmaf(dz, dz, fmaf(dy, dy, dx * dx));
                        if (idj == __float_as_int(qv.w) || (MI && idj < 0)) d2 = FAR_AWAY;
                        nearest = fminf(nearest, fabsf(d2 - p.r2_mid));
                        d2q[q] = d2;
                    }
                    if (__any_sync(FULL, nearest <= p.r2_band)) {
#pragma unroll
                        for (int q = 0; q < QB; ++q) {
                            if (q >= nq) break;
                            if (fabsf(d2q[q] - p.r2_mid) <= p.r2_band)
                                d2q[q] = exact_pair(p, __float_as_int(s_q[q].w), idj) ? fminf(d2q[q], p.r2_lo) : FAR_AWAY;
                        }
                    }
                    int mx = 0;
#pragma unroll
                    for (int q = 0; q < QB; ++q) {
                        if (q >= nq) break;
                        const bool ok = d2q[q] <= p.r2_lo;
                        const unsigned m = __ballot_sync(FULL, ok);
                        if (ok) list[q * MLP_QSTRIDE + qcnt[q] + __popc(m & lt_mask)] = cbase + lane;
                        qcnt[q] += __popc(m);
                        mx = qcnt[q] > mx ? qcnt[q] : mx;
                    }
                    return mx > MLP_QCAP - 32;
                };
                bool need = false;
                for (int cbase = 0;; cbase += 32) {
                    const bool done = cbase >= ns;
                    if (done || need) drain();
                    if (done) break;
                    need = phase_a(cbase);
                }
                if (!BWD && p.count && lane < nq) {
                    const int oq = __float_as_int(s_q[lane].w);
                    p.count[oq] = first_chunk ? s_tot[lane] : p.count[oq] + s_tot[lane];
                }
            }
            __syncwarp();
        };

        // the 27-cell stencil as candidate ranges (lane r < 27 resolves neighbour offset r)
        int r_cs = 0, r_ce = 0;
        float r_off[3] = {0.f, 0.f, 0.f};
        {
            const int off[3] = {lane % 3 - 1, (lane / 3) % 3 - 1, lane / 9 - 1};
            bool ok = lane < 27;
            int q[3] = {0, 0, 0};
            bool merged = false;
#pragma unroll
            for (int d = 0; d < 3; ++d) {
                if (p.nc[d] == 1) { ok = ok && off[d] == 0; r_off[d] = org[d]; continue; }
                if (d == 0 && c[0] >= 1 && c[0] <= p.nc[0] - 2) {
                    merged = true; ok = ok && off[0] == 0; q[0] = c[0] - 1; r_off[0] = org[0];
                    continue;
                }
                int v = c[d] + off[d];
                r_off[d] = org[d];
                if (v < 0) {
                    if (p.periodic[d]) { v += p.nc[d]; r_off[d] = org[d] + p.len[d]; }
                    else ok = false;
                } else if (v >= p.nc[d]) {
                    if (p.periodic[d]) { v -= p.nc[d]; r_off[d] = org[d] - p.len[d]; }
                    else ok = false;
                }
                q[d] = v;
            }
            if (ok) {
                const int id = (q[2] * p.nc[1] + q[1]) * p.nc[0] + q[0];
                r_cs = p.cell_start[id];
                r_ce = p.cell_start[id + (merged ? 3 : 1)];
            }
        }
        const int r_len = r_ce - r_cs;
        int r_incl = r_len;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(FULL, r_incl, o);
            if (lane >= o) r_incl += t;
        }
        const int total = __shfl_sync(FULL, r_incl, 31);
        // bounding box of the cell's own points (local coordinates), one register per lane: a candidate
        // farther than the cutoff from it is no neighbour of any of them and is not staged
        float bb;
        {
            float blo[3] = {FAR_AWAY, FAR_AWAY, FAR_AWAY}, bhi[3] = {-FAR_AWAY, -FAR_AWAY, -FAR_AWAY};
            for (int q = qs0 + lane; q < qe0; q += 32) {
                const float4 pq = p.spos[q];
                const float l[3] = {pq.x - org[0], pq.y - org[1], pq.z - org[2]};
#pragma unroll
                for (int d = 0; d < 3; ++d) { blo[d] = fminf(blo[d], l[d]); bhi[d] = fmaxf(bhi[d], l[d]); }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int d = 0; d < 3; ++d) {
                    blo[d] = fminf(blo[d], __shfl_xor_sync(FULL, blo[d], o));
                    bhi[d] = fmaxf(bhi[d], __shfl_xor_sync(FULL, bhi[d], o));
                }
            bb = lane == 0 ? blo[0] : lane == 1 ? blo[1] : lane == 2 ? blo[2] : lane == 3 ? bhi[0] : lane == 4 ? bhi[1] : bhi[2];
            if (mi0 && (lane == 0 || lane == 3)) bb = lane == 0 ? -FAR_AWAY : FAR_AWAY;   // a dimension folded by the explicit
            if (mi1 && (lane == 1 || lane == 4)) bb = lane == 1 ? -FAR_AWAY : FAR_AWAY;   // minimum image is not pruned
            if (mi2 && (lane == 2 || lane == 5)) bb = lane == 2 ? -FAR_AWAY : FAR_AWAY;
        }
        bool first_chunk = true;
        for (int lo = 0; lo < total || first_chunk; lo += MLP_STAGE_CAP) {
            const int ns = total - lo < MLP_STAGE_CAP ? total - lo : MLP_STAGE_CAP;
            int nst = 0;                                                     // candidates kept (warp uniform)
            constexpr int SU = 4;                                            // staging groups in flight
            for (int k0 = 0; k0 < ns; k0 += 32 * SU) {
                float4 c4[SU];
                float ox[SU], oy[SU], oz[SU];
#pragma unroll
                for (int u = 0; u < SU; ++u) {                               // all loads of the step first
                    const int k = k0 + 32 * u + lane;
                    const int v = lo + k;
                    int r = 0;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const int probe = __shfl_sync(FULL, r_incl, r + o - 1);
                        if (probe <= v) r += o;
                    }
                    r = r > 31 ? 31 : r;
                    const int src = __shfl_sync(FULL, r_cs, r) + (v - (__shfl_sync(FULL, r_incl, r) - __shfl_sync(FULL, r_len, r)));
                    ox[u] = __shfl_sync(FULL, r_off[0], r); oy[u] = __shfl_sync(FULL, r_off[1], r); oz[u] = __shfl_sync(FULL, r_off[2], r);
                    c4[u] = k < ns ? __ldg(p.spos + checked(src, p.n, CHECK_SLOT)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                const float lx = __shfl_sync(FULL, bb, 0), ly = __shfl_sync(FULL, bb, 1), lz = __shfl_sync(FULL, bb, 2);
                const float hx = __shfl_sync(FULL, bb, 3), hy = __shfl_sync(FULL, bb, 4), hz = __shfl_sync(FULL, bb, 5);
#pragma unroll
                for (int u = 0; u < SU; ++u) {
                    if (k0 + 32 * u >= ns) break;
                    const float4 val = make_float4(c4[u].x - ox[u], c4[u].y - oy[u], c4[u].z - oz[u], c4[u].w);
                    const float ex = fmaxf(fmaxf(lx - val.x, val.x - hx), 0.f);
                    const float ey = fmaxf(fmaxf(ly - val.y, val.y - hy), 0.f);
                    const float ez = fmaxf(fmaxf(lz - val.z, val.z - hz), 0.f);
                    const bool keep = k0 + 32 * u + lane < ns && fmaf(ez, ez, fmaf(ey, ey, ex * ex)) <= p.r2_hi * 1.0001f;
                    const unsigned m = __ballot_sync(FULL, keep);
                    if (keep) stage[nst + __popc(m & lt_mask)] = val;
                    nst += __popc(m);
                }
            }
            __syncwarp();
            process_chunk(nst, first_chunk);
            first_chunk = false;
        }
    }

    if constexpr (BWD) {
        // warps -> CTA copy in shared memory -> one atomic per parameter entry and CTA
        float* gW1s = sG;
        float* gb1s = gW1s + HID * MLP_DIN;
        float* gW2s = gb1s + HID;
        float* gb2s = gW2s + 4 * HID;
#pragma unroll
        for (int i = 0; i < HID / 2; ++i) atomicAdd(gW1s + (a0 + 2 * i) * MLP_DIN + k1, gW1acc[i]);
        if (lane < HID) {
#pragma unroll
            for (int o = 0; o < 4; ++o) atomicAdd(gW2s + o * HID + lane, gW2acc[o]);
            atomicAdd(gb1s + lane, gb1acc);
        }
        if (lane < 4) atomicAdd(gb2s + lane, gb2acc);
        __syncthreads();
        for (int e = threadIdx.x; e < HID * MLP_DIN; e += TRAV_THREADS) {
            const int a = e / MLP_DIN, k = e % MLP_DIN;
            if (k < K && p.gW1) atomicAdd(p.gW1 + a * K + k, gW1s[e]);
        }
        for (int e = threadIdx.x; e < HID; e += TRAV_THREADS) if (p.gb1) atomicAdd(p.gb1 + e, gb1s[e]);
        for (int e = threadIdx.x; e < Fout * HID; e += TRAV_THREADS) if (p.gW2) atomicAdd(p.gW2 + e, gW2s[e]);
        if (threadIdx.x < Fout && p.gb2) atomicAdd(p.gb2 + threadIdx.x, gb2s[threadIdx.x]);
    }
}

template <int HID, int KQ, bool BWD, bool MI>
static tiga_status launch_mlp_t(const RadiusParams& p, cudaStream_t s) {
    using SM = MlpSmem<HID, BWD>;
    auto kern = radius_mlp_kernel<HID, KQ, BWD, MI>;
    if (SM::TOTAL > 48 * 1024) TIGA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SM::TOTAL));
    long long blocks = (p.ncells + TRAV_WARPS - 1) / TRAV_WARPS;
    const long long cap = 148LL * mlp_ctas_per_sm<HID, BWD>();       // persistent: parameter gradients are folded once per CTA
    if (blocks > cap) blocks = cap;
    kern<<<counted((unsigned)blocks), TRAV_THREADS, SM::TOTAL, s>>>(p);
    return launch_status();
}

template <int HID, bool BWD, bool MI>
static tiga_status launch_mlp_k(const RadiusParams& p, cudaStream_t s) {
    switch ((3 + p.Fin + 3) / 4) {
        case 1: return launch_mlp_t<HID, 1, BWD, MI>(p, s);
        case 2: return launch_mlp_t<HID, 2, BWD, MI>(p, s);
        case 3: return launch_mlp_t<HID, 3, BWD, MI>(p, s);
        default: return launch_mlp_t<HID, 4, BWD, MI>(p, s);
    }
}

template <bool BWD>
static tiga_status launch_mlp(const RadiusParams& p, int hidden, cudaStream_t s) {
    bool mi = false;
    for (int d = 0; d < 3; ++d) mi = mi || (p.periodic[d] && p.nc[d] == 1);
    if (hidden == 8) return mi ? launch_mlp_k<8, BWD, true>(p, s) : launch_mlp_k<8, BWD, false>(p, s);
    if (hidden == 16) return mi ? launch_mlp_k<16, BWD, true>(p, s) : launch_mlp_k<16, BWD, false>(p, s);
    return mi ? launch_mlp_k<32, BWD, true>(p, s) : launch_mlp_k<32, BWD, false>(p, s);
}

static tiga_status mlp_common(RadiusParams* p, const float* pos, const float* feat, int64_t n, float r, const tiga_box* box,
                              const tiga_edge_mlp* mlp, void* ws, size_t ws_bytes, int32_t** fill, RadiusLayout* lay) {
    if (!mlp) return TIGA_ERR_INVALID_ARG;
    if (mlp->f_in < 1 || mlp->f_out < 1 || mlp->hidden < 1) return TIGA_ERR_INVALID_ARG;
    if (mlp->f_in > 13 || mlp->f_out > 4 || (mlp->hidden != 8 && mlp->hidden != 16 && mlp->hidden != 32)) return TIGA_ERR_UNSUPPORTED;
    if (!mlp->W1 || !mlp->b1 || !mlp->W2 || !mlp->b2) return TIGA_ERR_INVALID_ARG;
    tiga_status st = fill_params(p, n, r, box);
    if (st != TIGA_OK) return st;
    if (n > 0 && (!pos || !aligned16(pos) || !feat || !aligned16(feat))) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_radius_workspace_bytes(n, mlp->f_in, r, box, 0)) return TIGA_ERR_WORKSPACE;
    *lay = carve_radius(p, ws, fill);
    p->pos = pos; p->feat = feat; p->F = mlp->f_in; p->Fin = mlp->f_in; p->Fout = mlp->f_out;
    p->W1 = mlp->W1; p->b1 = mlp->b1; p->W2 = mlp->W2; p->b2 = mlp->b2;
    return TIGA_OK;
}

}  // namespace tiga

using namespace tiga;

extern "C" tiga_status tiga_apply_radius_mlp(const float* pos, const float* feat, int64_t n, float r, const tiga_box* box,
                                             const tiga_edge_mlp* mlp, float* out, int32_t* count,
                                             void* ws, size_t ws_bytes, void* stream) {
    RadiusParams p{};
    int32_t* fill;
    RadiusLayout lay;
    tiga_status st = mlp_common(&p, pos, feat, n, r, box, mlp, ws, ws_bytes, &fill, &lay);
    if (st != TIGA_OK) return st;
    if (n == 0) return TIGA_OK;
    if (!out || !aligned16(out)) return TIGA_ERR_INVALID_ARG;
    p.out = out; p.count = count;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = run_binning(p, fill, lay.nblocks, s);
    if (st != TIGA_OK) return st;
    return launch_mlp<false>(p, mlp->hidden, s);
}

extern "C" tiga_status tiga_apply_radius_mlp_backward(const float* pos, const float* feat, int64_t n, float r, const tiga_box* box,
                                                      const tiga_edge_mlp* mlp, const float* grad_out,
                                                      float* grad_feat, float* grad_pos,
                                                      float* grad_W1, float* grad_b1, float* grad_W2, float* grad_b2,
                                                      void* ws, size_t ws_bytes, int reuse_plan, void* stream) {
    RadiusParams p{};
    int32_t* fill;
    RadiusLayout lay;
    tiga_status st = mlp_common(&p, pos, feat, n, r, box, mlp, ws, ws_bytes, &fill, &lay);
    if (st != TIGA_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int K = 3 + mlp->f_in;
    if (grad_W1) TIGA_CUDA_TRY(cudaMemsetAsync(grad_W1, 0, sizeof(float) * mlp->hidden * K, s));
    if (grad_b1) TIGA_CUDA_TRY(cudaMemsetAsync(grad_b1, 0, sizeof(float) * mlp->hidden, s));
    if (grad_W2) TIGA_CUDA_TRY(cudaMemsetAsync(grad_W2, 0, sizeof(float) * mlp->f_out * mlp->hidden, s));
    if (grad_b2) TIGA_CUDA_TRY(cudaMemsetAsync(grad_b2, 0, sizeof(float) * mlp->f_out, s));
    if (n == 0) return TIGA_OK;
    if (!grad_out || !aligned16(grad_out)) return TIGA_ERR_INVALID_ARG;
    p.gy = grad_out; p.gfeat = grad_feat; p.gpos = grad_pos;
    p.gW1 = grad_W1; p.gb1 = grad_b1; p.gW2 = grad_W2; p.gb2 = grad_b2;
    if (!reuse_plan) {
        st = run_binning(p, fill, lay.nblocks, s);
        if (st != TIGA_OK) return st;
    }
    return launch_mlp<true>(p, mlp->hidden, s);
}

namespace tiga { unsigned check_status_radius_mlp(bool reset) { return read_check_status(reset); } }
