// Lennard-Jones message over the generated radius relation (fused cell-list traversal, paper
// Section 4.9), evaluated once per unordered pair.
//
// The pair force is antisymmetric and the pair energy symmetric, so the row sums
//     F_i = sum over j in N(i) of f_ij,   e_i = sum over j in N(i) of u_ij / 2
// can be formed by visiting every unordered pair {i, j} once and adding f_ij to row i and -f_ij
// to row j.  One warp owns a cell and tests its points against the points of the cell itself
// (each pair once, by index order) and of the 13 neighbour cells whose offset is lexicographically
// positive; the other 13 cells visit this one from their side.  That halves the candidate tests,
// the staging and the force evaluations of a traversal that walks all 27 cells per row.
//
// The price is that a row is no longer summed by a single warp: contributions arrive through
// 128-bit vector atomics (out must start at zero), so the summation order, and with it the last
// bits of the result, can change from run to run.  Neighbour counts are integers and stay exact.
//
// Structure inside a warp: the half stencil is staged in shared memory in the points' ORIGINAL
// coordinates; a cell whose stencil wraps around a periodic face moves the points next to the upper
// face down by the box length, which is exact in fp32, so a displacement is one rounded subtraction
// of two stored coordinates -- accurate to half an ulp of the displacement itself, however close the
// pair and however large the cell.  Candidates farther than the cutoff from the bounding box of the
// cell's points are dropped, phase A tests one staged candidate per lane against four queries and
// compacts accepted pairs into per-query lists by ballots (pairs within the fp32 error band of the
// cutoff are decided in fp64), phase B gives every query eight lanes that evaluate its listed pairs.
// (Evaluating the message for every tested pair with rejected weights forced to zero, without lists,
// was built and measured: the same instruction count at lower occupancy, 1.71 against 1.62 ms.)
#include "radius_shared.cuh"
#include <type_traits>

namespace tiga {

constexpr int LJ_STAGE_CAP = 256;
constexpr int LJ_QCAP = 64;
constexpr int LJ_QSTRIDE = LJ_QCAP + 1;
constexpr int LJ_STAGE_BYTES = (LJ_STAGE_CAP + STAGE_PAD) * 16;
constexpr int LJQ = 4;                        // queries per batch in this kernel
constexpr int LJ_LPQ = 32 / LJQ;              // lanes that share a query's list in phase B
constexpr int LJ_LIST_BYTES = (LJQ * LJ_QSTRIDE * 8 + 15) / 16 * 16;
constexpr int LJ_MISC_BYTES = LJQ * 16 + 3 * LJQ * 4 + LJQ * 4 + 32;        // queries, their coordinates by component, list lengths, the cell's frame
constexpr int LJ_PER_WARP = (LJ_STAGE_BYTES + LJ_LIST_BYTES + LJ_MISC_BYTES + 15) / 16 * 16;

// One warp, one cell; of a cell with more than QDENSE points only QSLICE as queries (from `first`): what such a cell
// leaves waits in the binning's queue of slices, which a second launch walks (QUEUE = true).
template <bool MI, bool COUNT, bool QUEUE>
__device__ __forceinline__ void lj_slice(const RadiusParams& p, const int cellid, const int first, unsigned char* s_raw) {
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    unsigned char* base = s_raw + (size_t)wib * LJ_PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);                                   // x, y, z in the frame of this cell, point id
    float2* list = reinterpret_cast<float2*>(base + LJ_STAGE_BYTES);                   // (stage slot, d2) per query
    float4* s_q = reinterpret_cast<float4*>(base + LJ_STAGE_BYTES + LJ_LIST_BYTES);
    float* s_qc = reinterpret_cast<float*>(s_q + LJQ);        // x[LJQ], y[LJQ], z[LJQ]: read two queries at a time
    int* s_n = reinterpret_cast<int*>(s_qc + 3 * LJQ);
    float* s_frame = reinterpret_cast<float*>(s_n + LJQ);     // thresholds [3], shifts [3] (kept out of the registers)

    const int c[3] = {cellid % p.nc[0], (cellid / p.nc[0]) % p.nc[1], cellid / (p.nc[0] * p.nc[1])};
    // a periodic dimension with three cells or fewer has no consistent shifted frame: explicit minimum image
    const bool mi0 = MI && p.periodic[0] && p.nc[0] <= 3, mi1 = MI && p.periodic[1] && p.nc[1] <= 3, mi2 = MI && p.periodic[2] && p.nc[2] <= 3;
    const float half0 = 0.5f * p.len[0], half1 = 0.5f * p.len[1], half2 = 0.5f * p.len[2];
    const unsigned lt_mask = (1u << lane) - 1u;
    float4* out4 = reinterpret_cast<float4*>(p.out);

    // displacement query - candidate of two points in the cell's frame
    auto delta = [&](const float4& q, const float4& c4, float& dx, float& dy, float& dz) {
        dx = (MI && mi0) ? mi_delta(q.x, c4.x, p.len[0], half0) : q.x - c4.x;
        dy = (MI && mi1) ? mi_delta(q.y, c4.y, p.len[1], half1) : q.y - c4.y;
        dz = (MI && mi2) ? mi_delta(q.z, c4.z, p.len[2], half2) : q.z - c4.z;
    };
    // frame of this cell: in a dimension whose stencil wraps around a face, every coordinate above the
    // threshold moves down by the box length (the wrapped cell at the top when the cell touches the lower
    // face; the cell and its lower neighbour when it touches the upper face).  Both shifts are exact.
    bool face = false;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        float thr = FAR_AWAY;
        if (p.periodic[d] && p.nc[d] >= 4) {
            if (c[d] == 0) { thr = 2.5f * p.hcell[d]; face = true; }
            else if (c[d] == p.nc[d] - 1) { thr = 1.5f * p.hcell[d]; face = true; }
        }
        if (lane == d) { s_frame[d] = thr; s_frame[3 + d] = p.len[d]; }
    }
    __syncwarp();
    auto to_frame = [&](float4 v) -> float4 {
        if (face) {
            if (v.x > s_frame[0]) v.x -= s_frame[3];
            if (v.y > s_frame[1]) v.y -= s_frame[4];
            if (v.z > s_frame[2]) v.z -= s_frame[5];
        }
        return v;
    };

    // ---- half stencil: lane 0 is the cell itself, lanes 1..13 the lexicographically positive offsets
    int r_cs = 0, r_len = 0;
    {
        const int L = 13 + lane;
        const int off[3] = {L % 3 - 1, (L / 3) % 3 - 1, L / 9 - 1};
        bool ok = lane < 14;
        int q[3] = {0, 0, 0};
#pragma unroll
        for (int d = 0; d < 3; ++d) {
            if (p.nc[d] == 1) { ok = ok && off[d] == 0; continue; }
            int v = c[d] + off[d];
            if (v < 0) { if (p.periodic[d]) v += p.nc[d]; else ok = false; }
            else if (v >= p.nc[d]) { if (p.periodic[d]) v -= p.nc[d]; else ok = false; }
            q[d] = v;
        }
        if (ok) {
            const int id = (q[2] * p.nc[1] + q[1]) * p.nc[0] + q[0];
            r_cs = p.cell_start[id];
            r_len = p.cell_start[id + 1] - r_cs;
        }
    }
    // lane 0 resolved the cell itself: its run is the cell's own points (one load round trip fewer
    // than asking for them first)
    const int own0 = __shfl_sync(FULL, r_cs, 0), nown = __shfl_sync(FULL, r_len, 0);
    if (nown == 0) return;
    const int qs0 = own0 + first, qe0 = nown > QDENSE ? slice_end(qs0, own0 + nown) : own0 + nown;     // this warp's queries
    int r_incl = r_len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, r_incl, o);
        if (lane >= o) r_incl += t;
    }
    const int total = __shfl_sync(FULL, r_incl, 31);

    // flattened stencil position v -> its run and address in the cell-ordered points
    auto locate = [&](const int v, int& run) -> int {
        int r = 0;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {                 // 14 runs: a four-step search
            const int probe = __shfl_sync(FULL, r_incl, r + o - 1);
            if (probe <= v) r += o;
        }
        run = r > 13 ? 13 : r;
        return __shfl_sync(FULL, r_cs, run) + (v - (__shfl_sync(FULL, r_incl, run) - __shfl_sync(FULL, r_len, run)));
    };
    constexpr int SU = 4;                                 // staging groups in flight
    // start fetching the first staging groups now: they arrive while the bounding box is formed
#pragma unroll
    for (int u = 0; u < SU; ++u) {
        int run;
        const int v = 32 * u + lane;
        const int src = locate(v, run);
        if (v < total) asm volatile("prefetch.global.L1 [%0];" ::"l"(p.spos + src));
    }

    // ---- bounding box of the cell's own points in the cell's frame, one register per lane
    float bb;
    {
        float blo[3] = {FAR_AWAY, FAR_AWAY, FAR_AWAY}, bhi[3] = {-FAR_AWAY, -FAR_AWAY, -FAR_AWAY};
        for (int q = qs0 + lane; q < qe0; q += 32) {
            const float4 pq = to_frame(p.spos[q]);
            const float l[3] = {pq.x, pq.y, pq.z};
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

    const float s2 = p.p1 * p.p1, e24 = 24.f * p.p0, e2x = 2.f * p.p0;

    // ---- all queries of the cell against the ns staged candidates; the first nself of them are the
    //      cell's own points, in the same order as the queries
    auto process_chunk = [&](const int ns, const int nself) {
        if (lane < STAGE_PAD) stage[ns + lane] = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-1));
        for (int qb0 = qs0; qb0 < qe0; qb0 += LJQ) {
            const int nq = (qe0 - qb0 < LJQ) ? qe0 - qb0 : LJQ;
            __syncwarp();
            if (lane < LJQ) {
                // absent queries of a short batch sit far away: whatever is computed for them is never used
                float4 lq4 = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-2));
                if (lane < nq) lq4 = to_frame(p.spos[qb0 + lane]);
                s_q[lane] = lq4;
                s_qc[lane] = lq4.x; s_qc[LJQ + lane] = lq4.y; s_qc[2 * LJQ + lane] = lq4.z;
            }
            __syncwarp();
            int qcnt[LJQ];
#pragma unroll
            for (int q = 0; q < LJQ; ++q) qcnt[q] = 0;

            auto drain = [&]() {
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int q = 0; q < LJQ; ++q) s_n[q] = qcnt[q];
                }
                __syncwarp();
                const int q = lane / LJ_LPQ, sub = lane % LJ_LPQ;
                float fx = 0.f, fy = 0.f, fz = 0.f, en = 0.f;
                int n = 0;
                if (q < nq) {
                    const float4 qv = s_q[q];
                    n = s_n[q];
                    const float2* lq = list + q * LJ_QSTRIDE;
                    for (int t = sub; t < n; t += 2 * LJ_LPQ) {
                        float2 e[2];
                        float4 pj[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            e[u] = lq[t + LJ_LPQ * u < n ? t + LJ_LPQ * u : t];
                            pj[u] = stage[__float_as_int(e[u].x)];
                        }
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            // the arithmetic runs for both slots of the step; an absent pair has inv = 0
                            // (zero force and energy) and only its atomics are switched off
                            const bool valid = t + LJ_LPQ * u < n;
                            const float inv = valid ? fast_rcp(e[u].y) : 0.f;
                            const float qq = s2 * inv;
                            const float q3 = qq * qq * qq;
                            const float fs = e24 * (2.f * q3 * q3 - q3) * inv;
                            const float ee = e2x * (q3 * q3 - q3);
                            float dx, dy, dz;
                            delta(qv, pj[u], dx, dy, dz);
                            const float gx = fs * dx, gy = fs * dy, gz = fs * dz;
                            fx += gx; fy += gy; fz += gz; en += ee;
                            const int idj = __float_as_int(pj[u].w);
                            if (valid) {
                                const int row_j = checked(idj, p.n, CHECK_POINT);
                                atomicAdd(out4 + row_j, make_float4(-gx, -gy, -gz, ee));    // the pair's other row
                                if (COUNT) atomicAdd(p.count + row_j, 1);
                            }
                        }
                    }
                }
#pragma unroll
                for (int o = 1; o < LJ_LPQ; o <<= 1) {
                    fx += __shfl_xor_sync(FULL, fx, o); fy += __shfl_xor_sync(FULL, fy, o);
                    fz += __shfl_xor_sync(FULL, fz, o); en += __shfl_xor_sync(FULL, en, o);
                }
                if (q < nq && sub == 0 && n > 0) {
                    const int idq = checked(__float_as_int(s_q[q].w), p.n, CHECK_POINT);
                    atomicAdd(out4 + idq, make_float4(fx, fy, fz, en));
                    if (COUNT) atomicAdd(p.count + idq, n);
                }
#pragma unroll
                for (int q2 = 0; q2 < LJQ; ++q2) qcnt[q2] = 0;
                __syncwarp();
            };

            // ---- phase A: one staged candidate per lane against the queries of the batch.
            //      OWN: the group holds points of the cell itself, which pair only with later ones.
            auto phase_a = [&](const int cbase, auto full_batch, auto own_group) -> bool {
                constexpr bool FULLB = decltype(full_batch)::value;
                constexpr bool OWN = decltype(own_group)::value;
                const float4 pj = stage[cbase + lane];
                const int idj = __float_as_int(pj.w);
                const bool own = OWN && cbase + lane < nself;
                float d2q[LJQ];
                float nearest = FAR_AWAY;       // smallest |d2 - r^2| seen by this lane
                if constexpr (!MI) {
                    // squared distances of two queries per instruction (same operations and roundings as
                    // the scalar form: a product, then two fused multiply-adds)
                    const f32x2 px = pack2(pj.x, pj.x), py = pack2(pj.y, pj.y), pz = pack2(pj.z, pj.z);
                    const f32x2* qx2 = reinterpret_cast<const f32x2*>(s_qc);
#pragma unroll
                    for (int h = 0; h < LJQ / 2; ++h) {
                        if (!FULLB && 2 * h >= nq) break;
                        const f32x2 dx = sub2(qx2[h], px), dy = sub2(qx2[LJQ / 2 + h], py), dz = sub2(qx2[LJQ + h], pz);
                        unpack2(fma2(dz, dz, fma2(dy, dy, mul2(dx, dx))), d2q[2 * h], d2q[2 * h + 1]);
                    }
#pragma unroll
                    for (int q = 0; q < LJQ; ++q) {
                        if (!FULLB && q >= nq) break;
                        if (OWN && own && idj <= __float_as_int(s_q[q].w)) d2q[q] = FAR_AWAY;      // own cell: each pair once
                        nearest = fminf(nearest, fabsf(d2q[q] - p.r2_mid));
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < LJQ; ++q) {
                        if (!FULLB && q >= nq) break;
                        const float4 qv = s_q[q];
                        float dx, dy, dz;
                        delta(qv, pj, dx, dy, dz);
                        float d2 = fmaf(dz, dz, fmaf(dy, dy, dx * dx));
                        if (OWN && own && idj <= __float_as_int(qv.w)) d2 = FAR_AWAY;      // own cell: each pair once
                        if (idj < 0) d2 = FAR_AWAY;                                        // folded sentinels
                        nearest = fminf(nearest, fabsf(d2 - p.r2_mid));
                        d2q[q] = d2;
                    }
                }
                if (__any_sync(FULL, nearest <= p.r2_band)) {
                    // some pair lies within the fp32 error band of the cutoff: decide it in fp64
#pragma unroll
                    for (int q = 0; q < LJQ; ++q) {
                        if (!FULLB && q >= nq) break;
                        if (fabsf(d2q[q] - p.r2_mid) <= p.r2_band)
                            d2q[q] = exact_pair(p, __float_as_int(s_q[q].w), idj) ? fminf(d2q[q], p.r2_lo) : FAR_AWAY;
                    }
                }
                int mx = 0;
#pragma unroll
                for (int q = 0; q < LJQ; ++q) {
                    if (!FULLB && q >= nq) break;
                    const bool ok = d2q[q] <= p.r2_lo;
                    const unsigned m = __ballot_sync(FULL, ok);
                    float2* dst = list + q * LJ_QSTRIDE + qcnt[q] + __popc(m & lt_mask);
                    if (ok) *dst = make_float2(__int_as_float(cbase + lane), d2q[q]);
                    qcnt[q] += __popc(m);
                    mx = qcnt[q] > mx ? qcnt[q] : mx;
                }
                return mx > LJ_QCAP - 32;
            };

            bool need = false;
            for (int cbase = 0;; cbase += 32) {
                const bool done = cbase >= ns;
                if (done || need) drain();
                if (done) break;
                if (cbase < nself)
                    need = (nq == LJQ) ? phase_a(cbase, std::true_type{}, std::true_type{}) : phase_a(cbase, std::false_type{}, std::true_type{});
                else
                    need = (nq == LJQ) ? phase_a(cbase, std::true_type{}, std::false_type{}) : phase_a(cbase, std::false_type{}, std::false_type{});
            }
        }
        __syncwarp();
        __syncwarp();
    };

    // ---- flat staging of the kept candidates, a chunk at a time
    for (int lo = 0; lo < total; lo += LJ_STAGE_CAP) {
        const int nin = total - lo < LJ_STAGE_CAP ? total - lo : LJ_STAGE_CAP;
        int nst = 0;
        for (int k0 = 0; k0 < nin; k0 += 32 * SU) {
            float4 c4[SU];
#pragma unroll
            for (int u = 0; u < SU; ++u) {                // all loads of the step first
                const int k = k0 + 32 * u + lane;
                int run;
                const int src = locate(lo + k, run);
                c4[u] = k < nin ? __ldg(p.spos + checked(src, p.n, CHECK_SLOT)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const float lx = __shfl_sync(FULL, bb, 0), ly = __shfl_sync(FULL, bb, 1), lz = __shfl_sync(FULL, bb, 2);
            const float hx = __shfl_sync(FULL, bb, 3), hy = __shfl_sync(FULL, bb, 4), hz = __shfl_sync(FULL, bb, 5);
#pragma unroll
            for (int u = 0; u < SU; ++u) {
                if (k0 + 32 * u >= nin) break;
                const float4 val = to_frame(c4[u]);
                const float ex = fmaxf(fmaxf(lx - val.x, val.x - hx), 0.f);
                const float ey = fmaxf(fmaxf(ly - val.y, val.y - hy), 0.f);
                const float ez = fmaxf(fmaxf(lz - val.z, val.z - hz), 0.f);
                // the cell's own points are always kept (a slice's box does not cover all of them, and the
                // own-pair rule below goes by their position at the head of the stage)
                const int kk = k0 + 32 * u + lane;
                const bool keep = kk < nin && (lo + kk < nown || fmaf(ez, ez, fmaf(ey, ey, ex * ex)) <= p.r2_hi * 1.0001f);
                const unsigned m = __ballot_sync(FULL, keep);
                if (keep) stage[nst + __popc(m & lt_mask)] = val;
                nst += __popc(m);
            }
        }
        __syncwarp();
        // the cell's own points come first in the flattened stencil and are never dropped
        const int nself = lo < nown ? (nown - lo < LJ_STAGE_CAP ? nown - lo : LJ_STAGE_CAP) : 0;
        process_chunk(nst, nself);
    }
}

// QUEUE = false: warp w takes cell w.  QUEUE = true: the warps of a small grid walk the queued slices.
template <bool MI, bool COUNT, bool QUEUE>
__global__ void __launch_bounds__(TRAV_THREADS, COUNT ? 8 : 7) radius_lj_pairs_kernel(const __grid_constant__ RadiusParams p) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    const int w = blockIdx.x * TRAV_WARPS + (threadIdx.x >> 5);
    if constexpr (!QUEUE) {
        if (w < p.ncells) lj_slice<MI, COUNT, false>(p, w, 0, s_raw);
    } else {
        const int n = *p.q_count;
        for (int it = w; it < n; it += gridDim.x * TRAV_WARPS) {
            const int2 item = p.q_items[it];
            lj_slice<MI, COUNT, true>(p, item.x, item.y, s_raw);
            __syncwarp();
        }
    }
}

template <bool MI, bool COUNT>
static tiga_status launch_lj_t(const RadiusParams& p, cudaStream_t s) {
    constexpr int smem = LJ_PER_WARP * TRAV_WARPS;
    auto kern = radius_lj_pairs_kernel<MI, COUNT, false>;
    auto kq = radius_lj_pairs_kernel<MI, COUNT, true>;
    if (smem > 48 * 1024) {
        TIGA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        TIGA_CUDA_TRY(cudaFuncSetAttribute(kq, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    }
    return two_passes(p, s, [&](const RadiusParams& q, unsigned grid) {
        if (q.q_mode) kq<<<counted(grid), TRAV_THREADS, smem, s>>>(q);
        else kern<<<counted(grid), TRAV_THREADS, smem, s>>>(q);
    });
}

tiga_status launch_lj_pairs(const RadiusParams& p, cudaStream_t s) {
    // rows are accumulated by atomics from several warps: start from zero
    TIGA_CUDA_TRY(cudaMemsetAsync(p.out, 0, (size_t)p.n * 4 * sizeof(float), s));
    if (p.count) TIGA_CUDA_TRY(cudaMemsetAsync(p.count, 0, (size_t)p.n * sizeof(int32_t), s));
    bool mi = false;
    for (int d = 0; d < 3; ++d) mi = mi || (p.periodic[d] && p.nc[d] <= 3);
    if (p.count) return mi ? launch_lj_t<true, true>(p, s) : launch_lj_t<false, true>(p, s);
    return mi ? launch_lj_t<true, false>(p, s) : launch_lj_t<false, false>(p, s);
}

}  // namespace tiga

namespace tiga { unsigned check_status_radius_lj(bool reset) { return read_check_status(reset); } }
