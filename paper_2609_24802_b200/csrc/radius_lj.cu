// Lennard-Jones message over the generated radius relation (fused cell-list traversal, paper
// Section 4.9), evaluated once per unordered pair, without pair lists.
//
// The pair force is antisymmetric and the pair energy symmetric, so the row sums
//     F_i = sum over j in N(i) of f_ij,   e_i = sum over j in N(i) of u_ij / 2
// can be formed by visiting every unordered pair {i, j} once and adding f_ij to row i and -f_ij
// to row j.  One warp owns a cell and tests its points against the points of the cell itself
// (each pair once, by index order) and of the 13 neighbour cells whose offset is lexicographically
// positive; the other 13 cells visit this one from their side.
//
// Inside a warp:
//   staging : the half stencil's candidates are copied into shared memory in their ORIGINAL
//             coordinates; a cell whose stencil wraps around a periodic face moves the points next to
//             the upper face down by the box length, which is exact in fp32.  A displacement is then
//             one rounded subtraction of two stored coordinates -- accurate to half an ulp of the
//             displacement itself, however close the pair and however large the cell.  Candidates
//             farther than the cutoff from the bounding box of the cell's own points are dropped.
//   pairs   : every lane keeps one staged candidate and meets a batch of four queries.  The message
//             is cheap (a reciprocal and a dozen multiplies), so it is evaluated for every tested pair
//             with the weight of a rejected pair forced to zero, two queries per packed fp32
//             instruction; nothing is compacted, listed or drained.  The query's row accumulates in
//             registers over all candidates (summed over the lanes once per batch), the candidate's
//             row in shared memory over all queries.  Pairs whose fp32 distance falls within a few ulps
//             of the cutoff are decided in fp64 with the defining formula.
//   output  : one 128-bit vector atomic per query and one per staged candidate that met a neighbour
//             (out starts at zero), instead of one per pair.  The summation order of a row depends
//             on scheduling, so the last bits can change from run to run; neighbour counts are exact.
#include "radius_shared.cuh"
#include <type_traits>

namespace tiga {

constexpr int LJ_STAGE_CAP = 192;             // candidates staged per chunk
constexpr int LJQ = 4;                        // queries per batch
constexpr int LJ_STAGE_BYTES = (LJ_STAGE_CAP + STAGE_PAD) * 16;
constexpr int LJ_ACC_BYTES = (LJ_STAGE_CAP + STAGE_PAD) * 16;                 // padding lanes add zeros behind the last candidate
constexpr int LJ_RED_BYTES = 4 * LJQ * 4 + LJQ * 16;                          // reduced row sums of a batch, the batch's queries
template <bool COUNT> struct LjSmem {
    static constexpr int CNT_BYTES = COUNT ? (LJ_STAGE_CAP + STAGE_PAD) * 4 : 0;
    static constexpr int PER_WARP = (LJ_STAGE_BYTES + LJ_ACC_BYTES + CNT_BYTES + LJ_RED_BYTES + 15) / 16 * 16;
};

static __device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { f32x2 r; asm("add.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }

// minimum-image displacement of two coordinates of a periodic dimension that is not split into
// enough cells for a frame shift: the subtraction that can lose bits (x near 0 against x near len)
// is replaced by an exact shift of the coordinate next to the upper face
static __device__ __forceinline__ float mi_delta(float a, float b, float len, float half) {
    float t = a - b;
    if (t > half) t = (a - len) - b;
    else if (t < -half) t = a - (b - len);
    return t;
}

template <bool MI, bool COUNT>
__global__ void __launch_bounds__(TRAV_THREADS, 5) radius_lj_pairs_kernel(const __grid_constant__ RadiusParams p) {
    constexpr unsigned FULL = 0xffffffffu;
    using SM = LjSmem<COUNT>;
    extern __shared__ __align__(16) unsigned char s_raw[];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int cellid = blockIdx.x * TRAV_WARPS + wib;
    if (cellid >= p.ncells) return;
    unsigned char* base = s_raw + (size_t)wib * SM::PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);                                   // x, y, z (frame of this cell), point id
    float4* acc = reinterpret_cast<float4*>(base + LJ_STAGE_BYTES);                    // the candidates' rows: -force, energy
    int* cnt = reinterpret_cast<int*>(base + LJ_STAGE_BYTES + LJ_ACC_BYTES);           // the candidates' neighbour counts
    float* s_red = reinterpret_cast<float*>(base + LJ_STAGE_BYTES + LJ_ACC_BYTES + SM::CNT_BYTES);    // [LJQ][4]
    float4* s_q = reinterpret_cast<float4*>(s_red + 4 * LJQ);

    const int c[3] = {cellid % p.nc[0], (cellid / p.nc[0]) % p.nc[1], cellid / (p.nc[0] * p.nc[1])};
    // a periodic dimension with three cells or fewer has no consistent shifted frame: explicit minimum image
    const bool mi0 = MI && p.periodic[0] && p.nc[0] <= 3, mi1 = MI && p.periodic[1] && p.nc[1] <= 3, mi2 = MI && p.periodic[2] && p.nc[2] <= 3;
    const unsigned lt_mask = (1u << lane) - 1u;
    float4* out4 = reinterpret_cast<float4*>(p.out);

    // frame of this cell: in a dimension whose stencil wraps around a face, every coordinate above the
    // threshold moves down by the box length (the wrapped cell at the top when the cell touches the lower
    // face; the cell and its lower neighbour when it touches the upper face).  Both shifts are exact.
    float thr[3];
    bool face = false;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        thr[d] = FAR_AWAY;
        if (p.periodic[d] && p.nc[d] >= 4) {
            if (c[d] == 0) { thr[d] = 2.5f * p.hcell[d]; face = true; }
            else if (c[d] == p.nc[d] - 1) { thr[d] = 1.5f * p.hcell[d]; face = true; }
        }
    }
    auto to_frame = [&](float4 v) -> float4 {
        if (face) {
            if (v.x > thr[0]) v.x -= p.len[0];
            if (v.y > thr[1]) v.y -= p.len[1];
            if (v.z > thr[2]) v.z -= p.len[2];
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
    const int qs0 = __shfl_sync(FULL, r_cs, 0), nown = __shfl_sync(FULL, r_len, 0), qe0 = qs0 + nown;
    if (nown == 0) return;
    int r_incl = r_len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, r_incl, o);
        if (lane >= o) r_incl += t;
    }
    const int total = __shfl_sync(FULL, r_incl, 31);

    // flattened stencil position v -> its address in the cell-ordered points
    auto locate = [&](const int v) -> int {
        int r = 0;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {                 // 14 runs: a four-step search
            const int probe = __shfl_sync(FULL, r_incl, r + o - 1);
            if (probe <= v) r += o;
        }
        r = r > 13 ? 13 : r;
        return __shfl_sync(FULL, r_cs, r) + (v - (__shfl_sync(FULL, r_incl, r) - __shfl_sync(FULL, r_len, r)));
    };
    constexpr int SU = 4;                                 // staging groups in flight
#pragma unroll
    for (int u = 0; u < SU; ++u) {
        const int v = 32 * u + lane;
        const int src = locate(v);
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

    const float ns2 = -(p.p1 * p.p1), e24 = 24.f * p.p0, e2x = 2.f * p.p0;
    const f32x2 ns2_2 = pack2(ns2, ns2), e24_2 = pack2(e24, e24), e2x_2 = pack2(e2x, e2x), two_2 = pack2(2.f, 2.f);
    const float half0 = 0.5f * p.len[0], half1 = 0.5f * p.len[1], half2 = 0.5f * p.len[2];

    // ---- all queries of the cell against the ns staged candidates; the first nself of them are points
    //      of the cell itself (they pair only with queries of a lower point id)
    auto process_chunk = [&](const int ns, const int nself) {
        // padding candidates sit far away on one side, absent queries of a short batch on the other
        if (lane < STAGE_PAD) stage[ns + lane] = make_float4(-FAR_AWAY, -FAR_AWAY, -FAR_AWAY, __int_as_float(-1));
        for (int k = lane; k < ns + STAGE_PAD; k += 32) {
            acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (COUNT) cnt[k] = 0;
        }
        for (int qb0 = qs0; qb0 < qe0; qb0 += LJQ) {
            const int nq = (qe0 - qb0 < LJQ) ? qe0 - qb0 : LJQ;
            __syncwarp();
            if (lane < LJQ) {
                float4 q4 = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(0x7fffffff));
                if (lane < nq) q4 = to_frame(p.spos[qb0 + lane]);
                s_q[lane] = q4;
            }
            __syncwarp();
            f32x2 qx[LJQ / 2], qy[LJQ / 2], qz[LJQ / 2];
            int idq[LJQ];
#pragma unroll
            for (int h = 0; h < LJQ / 2; ++h) {
                const float4 a = s_q[2 * h], b = s_q[2 * h + 1];
                qx[h] = pack2(a.x, b.x); qy[h] = pack2(a.y, b.y); qz[h] = pack2(a.z, b.z);
                idq[2 * h] = __float_as_int(a.w); idq[2 * h + 1] = __float_as_int(b.w);
            }
            f32x2 fx[LJQ / 2], fy[LJQ / 2], fz[LJQ / 2], en[LJQ / 2];      // the queries' rows, per lane
            int ci[LJQ];
#pragma unroll
            for (int h = 0; h < LJQ / 2; ++h) { fx[h] = fy[h] = fz[h] = en[h] = 0ull; }
#pragma unroll
            for (int q = 0; q < LJQ; ++q) ci[q] = 0;

            for (int cbase = 0; cbase < ns; cbase += 32) {
                const float4 pj = stage[cbase + lane];
                const int idj = __float_as_int(pj.w);
                // own cell: each pair once -- the candidate must have the higher point id (an absent
                // query's id is above every point id)
                const int idlim = cbase + lane < nself ? idj : 0x7fffffff;
                const f32x2 px = pack2(pj.x, pj.x), py = pack2(pj.y, pj.y), pz = pack2(pj.z, pj.z);
                f32x2 gx = 0ull, gy = 0ull, gz = 0ull, ge = 0ull;            // the candidate's row over this batch (two partial sums)
                int cj = 0;
#pragma unroll
                for (int h = 0; h < LJQ / 2; ++h) {
                    f32x2 dx, dy, dz;
                    if constexpr (!MI) {
                        dx = sub2(qx[h], px); dy = sub2(qy[h], py); dz = sub2(qz[h], pz);
                    } else {
                        float ax, bx, ay, by, az, bz;
                        unpack2(qx[h], ax, bx); unpack2(qy[h], ay, by); unpack2(qz[h], az, bz);
                        dx = mi0 ? pack2(mi_delta(ax, pj.x, p.len[0], half0), mi_delta(bx, pj.x, p.len[0], half0)) : sub2(qx[h], px);
                        dy = mi1 ? pack2(mi_delta(ay, pj.y, p.len[1], half1), mi_delta(by, pj.y, p.len[1], half1)) : sub2(qy[h], py);
                        dz = mi2 ? pack2(mi_delta(az, pj.z, p.len[2], half2), mi_delta(bz, pj.z, p.len[2], half2)) : sub2(qz[h], pz);
                    }
                    float d2a, d2b;
                    unpack2(fma2(dz, dz, fma2(dy, dy, mul2(dx, dx))), d2a, d2b);
                    bool oka = d2a <= p.r2_hi && idq[2 * h] < idlim;
                    bool okb = d2b <= p.r2_hi && idq[2 * h + 1] < idlim;
                    if (__any_sync(FULL, (oka && d2a > p.r2_lo) || (okb && d2b > p.r2_lo))) {
                        // some pair lies within the fp32 error band of the cutoff: decide it in fp64
                        if (oka && d2a > p.r2_lo) oka = exact_pair(p, idq[2 * h], idj);
                        if (okb && d2b > p.r2_lo) okb = exact_pair(p, idq[2 * h + 1], idj);
                    }
                    const f32x2 inv = pack2(oka ? fast_rcp(d2a) : 0.f, okb ? fast_rcp(d2b) : 0.f);
                    const f32x2 nqq = mul2(ns2_2, inv);                       // -(s/d)^2
                    const f32x2 nq3 = mul2(mul2(nqq, nqq), nqq);              // -(s/d)^6
                    const f32x2 t = mul2(nq3, nq3);                           // (s/d)^12
                    const f32x2 fs = mul2(fma2(t, two_2, nq3), mul2(e24_2, inv));     // 24 eps (2 (s/d)^12 - (s/d)^6) / d^2
                    const f32x2 ee = mul2(e2x_2, add2(t, nq3));               // half of the pair energy
                    fx[h] = fma2(fs, dx, fx[h]); fy[h] = fma2(fs, dy, fy[h]); fz[h] = fma2(fs, dz, fz[h]); en[h] = add2(en[h], ee);
                    gx = fma2(fs, dx, gx); gy = fma2(fs, dy, gy); gz = fma2(fs, dz, gz); ge = add2(ge, ee);
                    if (COUNT) {
                        ci[2 * h] += __popc(__ballot_sync(FULL, oka)); ci[2 * h + 1] += __popc(__ballot_sync(FULL, okb));
                        cj += (oka ? 1 : 0) + (okb ? 1 : 0);
                    }
                }
                float a0, a1, b0, b1, c0, c1, e0, e1;
                unpack2(gx, a0, a1); unpack2(gy, b0, b1); unpack2(gz, c0, c1); unpack2(ge, e0, e1);
                float4 g = acc[cbase + lane];
                g.x -= a0 + a1; g.y -= b0 + b1; g.z -= c0 + c1; g.w += e0 + e1;
                acc[cbase + lane] = g;
                if (COUNT) cnt[cbase + lane] += cj;
            }

            // ---- the queries' rows: 4 LJQ partial sums per lane -> one total each, by a halving exchange
            //      (a lane sends the half it gives up and keeps the half it owns), then one plain step
            float v[4 * LJQ];
#pragma unroll
            for (int h = 0; h < LJQ / 2; ++h) {
                unpack2(fx[h], v[8 * h + 0], v[8 * h + 4]); unpack2(fy[h], v[8 * h + 1], v[8 * h + 5]);
                unpack2(fz[h], v[8 * h + 2], v[8 * h + 6]); unpack2(en[h], v[8 * h + 3], v[8 * h + 7]);
            }
            // v[4 q + c]: component c of query q
            static_assert(LJQ == 4, "the exchange below reduces sixteen values");
            {
                const bool up = lane & 16;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float send = up ? v[k] : v[k + 8];
                    const float keep = up ? v[k + 8] : v[k];
                    v[k] = keep + __shfl_xor_sync(FULL, send, 16);
                }
            }
            {
                const bool up = lane & 8;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float send = up ? v[k] : v[k + 4];
                    const float keep = up ? v[k + 4] : v[k];
                    v[k] = keep + __shfl_xor_sync(FULL, send, 8);
                }
            }
            {
                const bool up = lane & 4;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const float send = up ? v[k] : v[k + 2];
                    const float keep = up ? v[k + 2] : v[k];
                    v[k] = keep + __shfl_xor_sync(FULL, send, 4);
                }
            }
            {
                const bool up = lane & 2;
                const float send = up ? v[0] : v[1];
                const float keep = up ? v[1] : v[0];
                v[0] = keep + __shfl_xor_sync(FULL, send, 2);
            }
            v[0] += __shfl_xor_sync(FULL, v[0], 1);
            // lane L now owns entry 8 bit4(L) + 4 bit3(L) + 2 bit2(L) + bit1(L)
            if (!(lane & 1)) s_red[((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1)] = v[0];
            __syncwarp();
            if (lane < nq) {
                const float4 tot = *reinterpret_cast<const float4*>(s_red + 4 * lane);
                const int id = __float_as_int(s_q[lane].w);
                if (tot.x != 0.f || tot.y != 0.f || tot.z != 0.f || tot.w != 0.f) atomicAdd(out4 + id, tot);
                if (COUNT) {
                    int mine = 0;
#pragma unroll
                    for (int q = 0; q < LJQ; ++q) mine = lane == q ? ci[q] : mine;
                    if (mine) atomicAdd(p.count + id, mine);
                }
            }
        }
        __syncwarp();
        // ---- the candidates' rows
        for (int k = lane; k < ns; k += 32) {
            const float4 g = acc[k];
            const int id = __float_as_int(stage[k].w);
            if (g.x != 0.f || g.y != 0.f || g.z != 0.f || g.w != 0.f) atomicAdd(out4 + id, g);
            if (COUNT) { const int n = cnt[k]; if (n) atomicAdd(p.count + id, n); }
        }
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
                const int src = locate(lo + k);
                c4[u] = k < nin ? __ldg(p.spos + src) : make_float4(0.f, 0.f, 0.f, 0.f);
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
                const bool keep = k0 + 32 * u + lane < nin && fmaf(ez, ez, fmaf(ey, ey, ex * ex)) <= p.r2_hi * 1.0001f;
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

template <bool MI, bool COUNT>
static tiga_status launch_lj_t(const RadiusParams& p, cudaStream_t s) {
    const unsigned blocks = (unsigned)((p.ncells + TRAV_WARPS - 1) / TRAV_WARPS);
    constexpr int smem = LjSmem<COUNT>::PER_WARP * TRAV_WARPS;
    auto kern = radius_lj_pairs_kernel<MI, COUNT>;
    if (smem > 48 * 1024) TIGA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    kern<<<counted(blocks), TRAV_THREADS, smem, s>>>(p);
    return launch_status();
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
