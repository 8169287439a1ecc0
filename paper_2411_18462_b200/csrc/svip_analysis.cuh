// The analysis quantities of a (target row, draft row) pair (Eq. 1-6, appendix B).
#pragma once

#include "svip_draft.cuh"

namespace svip {
// ------------------------------------------------------------------ analysis quantities of a row pair
//
// Eq. 1-6 and appendix B: for p = softmax(target row / T) and q = softmax(draft row / T),
//   beta = sum min(p, q),  H_q = -sum q ln q,  KL(q||p) = sum q (ln q - ln p),  H_qp = H_q + KL,
//   gamma = H_qp / H_q and the three lower bounds on beta.
// One kernel, one cluster per pair, two phases:
//   1. both rows are streamed together through the cp.async ring (the only read from HBM).  With
//      a = l * c - M (log2 units, M a reference near the row's maximum) the warp accumulates
//      Zp = sum 2^ap, Zq = sum 2^aq, Aq = sum 2^aq aq and D = sum 2^aq (aq - ap); from these
//      H_q = ln2 (log2 Zq - Aq / Zq) and KL = ln2 (D / Zq - log2 Zq + log2 Zp): no normaliser is
//      needed while streaming.  KL is accumulated as a sum of differences, not as a difference of
//      two entropies, so that it keeps its precision when p is close to q.
//   2. beta does need the normalisers: min(p, q) = 2^min(ap - log2 Zp, aq - log2 Zq), one more pass
//      over the two rows with one exponential per element.  The launch shape keeps the rows of all
//      resident clusters within L2 (clusters of several blocks for long rows), so this pass does not go
//      back to HBM.
// Segments whose fast sums are not finite (-inf / NaN logits, rows that start far below their
// maximum, vectors that stick out of the row) are summed again by an exact masking path.

struct PairArgs {
    const void* t_logits;
    long t_row_stride;
    const void* q_logits;
    long q_row_stride;
    int V;
    float c;
    float c_bound;
    float* out;   // [pairs][8]
    unsigned* status;
    const float2* p_stats;   // kGiven: (max logit, Z) of every target row
    const float2* q_stats;   // kGiven: ... of every draft row
};

// Partial sums of a warp segment: the target side relative to rn(mp * c), the draft side to rn(mq * c).
struct PairPartial {
    float mp, Zp;
    float mq, Zq, Aq, D;
};

// Moves a partial to the references (Mp, Mq) >= its own.
__device__ __forceinline__ void pair_rescale(PairPartial& t, float Mp, float Mq, float c) {
    float dp = 0.f;
    if (t.mp > neg_inf()) {
        dp = __fmul_rn(t.mp, c) - __fmul_rn(Mp, c);
        t.Zp = t.Zp > 0.f ? t.Zp * ex2_approx(fmaxf(dp, kArgFloor)) : 0.f;
    } else {
        t.Zp = 0.f;
    }
    if (t.mq > neg_inf() && t.Zq > 0.f) {
        const float dq = __fmul_rn(t.mq, c) - __fmul_rn(Mq, c);
        const float sq = ex2_approx(fmaxf(dq, kArgFloor));
        t.D = sq > 0.f ? sq * __fmaf_rn(dq - dp, t.Zq, t.D) : 0.f;   // D may be +inf (p masked where q is not)
        t.Aq = sq * __fmaf_rn(dq, t.Zq, t.Aq);
        t.Zq *= sq;
    } else {
        t.Zq = 0.f; t.Aq = 0.f; t.D = 0.f;
    }
    t.mp = Mp; t.mq = Mq;
}

// All lanes return the merge of the 32 lanes' partials.
__device__ __forceinline__ PairPartial pair_warp_merge(PairPartial t, float c) {
    const float Mp = warp_max(t.mp), Mq = warp_max(t.mq);
    pair_rescale(t, Mp, Mq, c);
    t.Zp = warp_sum(t.Zp); t.Zq = warp_sum(t.Zq); t.Aq = warp_sum(t.Aq); t.D = warp_sum(t.D);
    return t;
}

// Streams warp segment `seg` of the two rows together: vectors inside both rows go through the
// ring (four stages per row), the ones that stick out of a row are handed over masked to -inf by
// lane 0; rows of different 16-byte phase are read element by element.  f(x, d) gets the target and
// draft logits of one vector.  kBackward walks the segment from its end to its start: a second pass over
// rows that were just streamed then meets the most recently read lines first, which are the ones L2 still
// holds when the pairs of all resident clusters together exceed it.
template <int DT, bool kBackward = false, class F>
__device__ __forceinline__ void stream_pair(const RowGeom& g, const RowGeom& gq, const void* qrow, int seg, int lane,
                                            uint32_t slot0, F&& f) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    constexpr uint32_t kSlotStride = kThreads * 16;
    constexpr int kDepth = kStages / 2;
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    auto masked = [&](int vi) {
        float x[EPV], d[EPV];
        unpack_masked<DT>(ld_vec(g.base + vi), vi, g, x);
        if (gq.pre == g.pre) {
            unpack_masked<DT>(ld_vec(gq.base + vi), vi, gq, d);
        } else {
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                const int i = vi * EPV + j - g.pre;
                d[j] = (i >= 0 && i < g.V) ? ElemTraits<DT>::load_one(qrow, i) : neg_inf();
            }
        }
        f(x, d);
    };
    if (gq.pre != g.pre) {
        for (int vi = v_lo + lane; vi < v_hi; vi += 32) masked(vi);
        return;
    }
    const bool head_edge = g.pre > 0;
    const bool tail_edge = ((g.pre + g.V) % EPV) != 0;
    int i_lo = v_lo, i_hi = v_hi;
    if (head_edge && v_lo == 0 && v_hi > 0) i_lo = 1;
    if (tail_edge && v_hi == g.nvec && i_hi > i_lo) i_hi = g.nvec - 1;
    // lane's vectors: vi0 + 32 * dir * it, it = 0 .. n-1
    const int span = i_hi - i_lo;
    const int n = span > lane ? (span - lane + 31) >> 5 : 0;
    const int vi0 = kBackward ? i_hi - 1 - lane : i_lo + lane;
    constexpr int dir = kBackward ? -32 : 32;
    const uint4* st = g.base + vi0;
    const uint4* sq = gq.base + vi0;
#pragma unroll
    for (int s = 0; s < kDepth; ++s) {
        if (s < n) {
            cp_async16(slot0 + s * kSlotStride, st + dir * s);
            cp_async16(slot0 + (kDepth + s) * kSlotStride, sq + dir * s);
        }
        cp_async_commit();
    }
    for (int it = 0; it < n; ++it) {
        cp_async_wait<kDepth - 1>();
        const uint32_t sa = slot0 + (it & (kDepth - 1)) * kSlotStride;
        const uint4 rt = lds128(sa);
        const uint4 rq = lds128(sa + kDepth * kSlotStride);
        const int nx = it + kDepth;
        if (nx < n) {
            cp_async16(sa, st + dir * nx);
            cp_async16(sa + kDepth * kSlotStride, sq + dir * nx);
        }
        cp_async_commit();
        float x[EPV], d[EPV];
        ElemTraits<DT>::unpack(rt, x);
        ElemTraits<DT>::unpack(rq, d);
        f(x, d);
    }
    cp_async_wait<0>();
    if (lane == 0) {
        if (head_edge && v_lo == 0 && v_hi > 0) masked(0);
        if (tail_edge && v_hi == g.nvec && v_lo < v_hi && !(g.nvec == 1 && head_edge)) masked(g.nvec - 1);
    }
}

// Exact partial of a warp segment: maxima first, then the sums with -inf / NaN logits masked.
// With beta != NULL the row normalisers are known (kp = M_p + log2 Z_p, kq likewise, in log2 units) and
// *beta receives the segment's sum of min(p, q).
template <int DT>
__device__ __noinline__ PairPartial pair_segment_exact(const RowGeom& g, const RowGeom& gq, const void* qrow, int seg,
                                                       float c, int lane, float kp = 0.f, float kq = 0.f,
                                                       float* beta = nullptr) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    auto load = [&](int vi, float (&x)[EPV], float (&d)[EPV]) {
        unpack_masked<DT>(ld_vec(g.base + vi), vi, g, x);
        if (gq.pre == g.pre) {
            unpack_masked<DT>(ld_vec(gq.base + vi), vi, gq, d);
        } else {
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                const int i = vi * EPV + j - g.pre;
                d[j] = (i >= 0 && i < g.V) ? ElemTraits<DT>::load_one(qrow, i) : neg_inf();
            }
        }
#pragma unroll
        for (int j = 0; j < EPV; ++j) { x[j] = fmaxf(x[j], neg_inf()); d[j] = fmaxf(d[j], neg_inf()); }   // NaN -> -inf
    };
    PairPartial t;
    t.mp = neg_inf(); t.mq = neg_inf(); t.Zp = 0.f; t.Zq = 0.f; t.Aq = 0.f; t.D = 0.f;
    for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
        float x[EPV], d[EPV];
        load(vi, x, d);
#pragma unroll
        for (int j = 0; j < EPV; ++j) { t.mp = fmaxf(t.mp, x[j]); t.mq = fmaxf(t.mq, d[j]); }
    }
    t.mp = warp_max(t.mp); t.mq = warp_max(t.mq);
    const float Mp = __fmul_rn(t.mp, c), Mq = __fmul_rn(t.mq, c);
    float b = 0.f;
    for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
        float x[EPV], d[EPV];
        load(vi, x, d);
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            const bool hp = x[j] > neg_inf(), hq = d[j] > neg_inf();
            if (beta && hp && hq) b += ex2_approx(fminf(__fmaf_rn(x[j], c, -kp), __fmaf_rn(d[j], c, -kq)));
            const float ap = hp ? __fmaf_rn(x[j], c, -Mp) : neg_inf();
            if (hp) t.Zp += ex2_approx(fmaxf(ap, kArgFloor));
            if (hq) {
                const float aq = __fmaf_rn(d[j], c, -Mq);
                const float eq = ex2_approx(fmaxf(aq, kArgFloor));
                t.Zq += eq;
                if (eq > 0.f) {
                    t.Aq = __fmaf_rn(eq, aq, t.Aq);
                    t.D = __fmaf_rn(eq, aq - ap, t.D);      // +inf where the target masks a token the draft keeps
                }
            }
        }
    }
    t.Zp = warp_sum(t.Zp); t.Zq = warp_sum(t.Zq); t.Aq = warp_sum(t.Aq); t.D = warp_sum(t.D);
    if (beta) *beta = warp_sum(b);
    return t;
}

struct PairShared {
    PairPartial part[kWarps];
    float beta[kWarps];
    PairPartial row;
};

// kGiven: the caller holds the normalisers of both rows (the draft step and the threshold kernel write
// them), so everything, beta included, comes out of the one pass over HBM.
template <int DT, bool kGiven = false>
__global__ void __launch_bounds__(kThreads, 2) pair_stats_kernel(PairArgs a) {
    using E = ElemTraits<DT>;
    constexpr int EPV = E::kEPV;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int r = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ PairShared sh;
    extern __shared__ uint4 ring[];
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;

    pdl_launch_dependents();
    const char* trow = static_cast<const char*>(a.t_logits) + static_cast<size_t>(r) * a.t_row_stride * E::kBytes;
    const char* qrow = static_cast<const char*>(a.q_logits) + static_cast<size_t>(r) * a.q_row_stride * E::kBytes;
    const RowGeom gt = make_geom<DT>(trow, a.V, S * kWarps);
    const RowGeom gq = make_geom<DT>(qrow, a.V, S * kWarps);
    const int seg = rank * kWarps + warp;
    pdl_wait();

    PairPartial t;
    float beta = 0.f;
    if (kGiven) {
        // ---- single pass: the references are the rows' maxima, the normalisers are known
        const float2 ps = a.p_stats[r], qs = a.q_stats[r];
        const float Mp = __fmul_rn(ps.x, a.c), Mq = __fmul_rn(qs.x, a.c);
        const float rZp = 1.0f / ps.y, rZq = 1.0f / qs.y;
        const bool usable = ps.y > 0.f && qs.y > 0.f && fabsf(ps.x) <= kMaxLogit && fabsf(qs.x) <= kMaxLogit;
        const f32x2 c2 = pack2(a.c, a.c), nmp2 = pack2(-Mp, -Mp), nmq2 = pack2(-Mq, -Mq), m1 = pack2(-1.f, -1.f);
        const f32x2 rzp2 = pack2(rZp, rZp), rzq2 = pack2(rZq, rZq);
        f32x2 Aq2 = pack2(0.f, 0.f), D2 = Aq2;
        float b1 = 0.f;
        if (usable) {
            stream_pair<DT>(gt, gq, qrow, seg, lane, slot0, [&](const float (&x)[EPV], const float (&d)[EPV]) {
#pragma unroll
                for (int j = 0; j < EPV; j += 2) {
                    const f32x2 ap2 = fma2(pack2(x[j], x[j + 1]), c2, nmp2);
                    const f32x2 aq2 = fma2(pack2(d[j], d[j + 1]), c2, nmq2);
                    float a0, a1, b0v, b1v;
                    unpack2(ap2, a0, a1);
                    unpack2(aq2, b0v, b1v);
                    const f32x2 eq2 = pack2(ex2_approx(b0v), ex2_approx(b1v));
                    Aq2 = fma2(eq2, aq2, Aq2);
                    D2 = fma2(eq2, fma2(ap2, m1, aq2), D2);
                    float p0, p1, q0, q1;
                    unpack2(mul2(pack2(ex2_approx(a0), ex2_approx(a1)), rzp2), p0, p1);
                    unpack2(mul2(eq2, rzq2), q0, q1);
                    beta += fminf(p0, q0);
                    b1 += fminf(p1, q1);
                }
            });
        }
        float z0, z1;
        unpack2(Aq2, z0, z1); t.Aq = z0 + z1;
        unpack2(D2, z0, z1); t.D = z0 + z1;
        beta += b1;
        const bool bad = !usable || !(fabsf(t.Aq) <= 3.0e38f) || !(fabsf(t.D) <= 3.0e38f) || !(beta == beta);
        if (__any_sync(0xffffffffu, bad)) {
            t = pair_segment_exact<DT>(gt, gq, qrow, seg, a.c, lane, Mp + log2f(ps.y), Mq + log2f(qs.y), &beta);
            pair_rescale(t, fmaxf(ps.x, t.mp), fmaxf(qs.x, t.mq), a.c);     // to the rows' references
        } else {
            t.mp = ps.x; t.mq = qs.x;
            t.Aq = warp_sum(t.Aq); t.D = warp_sum(t.D);
            beta = warp_sum(beta);
        }
        t.Zp = 1.f; t.Zq = 1.f;      // stand-ins (the merge drops partials without mass); the given normalisers are used
    } else {
    // ---- phase 1: Zp, Zq, Aq, D of the warp's segment, relative to the largest logits among its first vectors
    {
        int v_lo, v_hi;
        seg_range(gt, seg, v_lo, v_hi);
        float fp = neg_inf(), fq = neg_inf();
        if (v_lo + lane < v_hi) {
            float x[EPV];
            unpack_masked<DT>(ld_stream(gt.base + v_lo + lane), v_lo + lane, gt, x);
            fp = vec_max<EPV>(x);
            if (gq.pre == gt.pre) {
                unpack_masked<DT>(ld_stream(gq.base + v_lo + lane), v_lo + lane, gq, x);
                fq = vec_max<EPV>(x);
            }
        }
        const float refp = warp_max(fp), refq = warp_max(fq);
        bool bad = !(fabsf(refp) <= kMaxLogit) || !(fabsf(refq) <= kMaxLogit);
        const float Mp = __fmul_rn(refp, a.c), Mq = __fmul_rn(refq, a.c);
        const f32x2 c2 = pack2(a.c, a.c), nmp2 = pack2(-Mp, -Mp), nmq2 = pack2(-Mq, -Mq), m1 = pack2(-1.f, -1.f);
        f32x2 Zp2 = pack2(0.f, 0.f), Zq2 = Zp2, Aq2 = Zp2, D2 = Zp2;
        float rp = neg_inf(), rq = neg_inf();
        if (!bad) {
            stream_pair<DT>(gt, gq, qrow, seg, lane, slot0, [&](const float (&x)[EPV], const float (&d)[EPV]) {
#pragma unroll
                for (int j = 0; j < EPV; j += 2) {
                    rp = max3(rp, x[j], x[j + 1]);
                    rq = max3(rq, d[j], d[j + 1]);
                    const f32x2 ap2 = fma2(pack2(x[j], x[j + 1]), c2, nmp2);
                    const f32x2 aq2 = fma2(pack2(d[j], d[j + 1]), c2, nmq2);
                    float a0, a1, b0, b1;
                    unpack2(ap2, a0, a1);
                    unpack2(aq2, b0, b1);
                    const f32x2 ep2 = pack2(ex2_approx(a0), ex2_approx(a1));
                    const f32x2 eq2 = pack2(ex2_approx(b0), ex2_approx(b1));
                    Zp2 = add2(Zp2, ep2);
                    Zq2 = add2(Zq2, eq2);
                    Aq2 = fma2(eq2, aq2, Aq2);
                    D2 = fma2(eq2, fma2(ap2, m1, aq2), D2);
                }
            });
        }
        float z0, z1;
        unpack2(Zp2, z0, z1); t.Zp = z0 + z1;
        unpack2(Zq2, z0, z1); t.Zq = z0 + z1;
        unpack2(Aq2, z0, z1); t.Aq = z0 + z1;
        unpack2(D2, z0, z1); t.D = z0 + z1;
        bad = bad || !(fabsf(t.Zp) <= 3.0e38f) || !(fabsf(t.Zq) <= 3.0e38f) || !(fabsf(t.Aq) <= 3.0e38f) ||
              !(fabsf(t.D) <= 3.0e38f);
        if (__any_sync(0xffffffffu, bad)) {
            t = pair_segment_exact<DT>(gt, gq, qrow, seg, a.c, lane);
        } else {
            // from the references to the segment's own maxima, as the exact path reports them
            t.mp = refp; t.mq = refq;
            const float mp = warp_max(rp), mq = warp_max(rq);
            pair_rescale(t, mp, mq, a.c);
            t.Zp = warp_sum(t.Zp); t.Zq = warp_sum(t.Zq); t.Aq = warp_sum(t.Aq); t.D = warp_sum(t.D);
        }
    }
    }
    if (lane == 0) { sh.part[warp] = t; sh.beta[warp] = beta; }
    cluster.sync();
    // every block merges all segments of the cluster in the same order: the same bits everywhere
    if (warp == 0) {
        const int nseg = S * kWarps;
        PairPartial m;
        m.mp = neg_inf(); m.mq = neg_inf(); m.Zp = 0.f; m.Zq = 0.f; m.Aq = 0.f; m.D = 0.f;
        PairPartial e[kSegPerLane];
        const int per = (nseg + 31) / 32;
#pragma unroll
        for (int k = 0; k < kSegPerLane; ++k) {
            const int s = lane * per + k;
            e[k] = m;
            if (k < per && s < nseg) e[k] = cluster.map_shared_rank(&sh, s / kWarps)->part[s % kWarps];
            m.mp = fmaxf(m.mp, e[k].mp); m.mq = fmaxf(m.mq, e[k].mq);
        }
        const float Mp = warp_max(m.mp), Mq = warp_max(m.mq);
#pragma unroll
        for (int k = 0; k < kSegPerLane; ++k) {
            pair_rescale(e[k], Mp, Mq, a.c);
            m.Zp += e[k].Zp; m.Zq += e[k].Zq; m.Aq += e[k].Aq; m.D += e[k].D;
        }
        m.mp = Mp; m.mq = Mq;
        m.Zp = warp_sum(m.Zp); m.Zq = warp_sum(m.Zq); m.Aq = warp_sum(m.Aq); m.D = warp_sum(m.D);
        if (lane == 0) sh.row = m;
    }
    __syncthreads();
    PairPartial R = sh.row;
    if (kGiven) {
        const float2 ps = a.p_stats[r], qs = a.q_stats[r];
        // the partials are relative to the given maxima (pair_rescale above brought stragglers there)
        R.mp = ps.x; R.Zp = ps.y; R.mq = qs.x; R.Zq = qs.y;
    }
    const bool ok = R.Zp > 0.f && R.Zq > 0.f && fabsf(R.mp) <= kMaxLogit && fabsf(R.mq) <= kMaxLogit;

    // ---- phase 2: beta = sum 2^min(ap - log2 Zp, aq - log2 Zq), the rows now come from L2
    if (!kGiven) {
    beta = 0.f;
    if (ok) {
        const float kp = __fmul_rn(R.mp, a.c) + log2f(R.Zp), kq = __fmul_rn(R.mq, a.c) + log2f(R.Zq);
        float b1 = 0.f;
        stream_pair<DT, true>(gt, gq, qrow, seg, lane, slot0, [&](const float (&x)[EPV], const float (&d)[EPV]) {
#pragma unroll
            for (int j = 0; j < EPV; j += 2) {
                const float l0 = fminf(__fmaf_rn(fmaxf(x[j], neg_inf()), a.c, -kp),
                                       __fmaf_rn(fmaxf(d[j], neg_inf()), a.c, -kq));
                const float l1 = fminf(__fmaf_rn(fmaxf(x[j + 1], neg_inf()), a.c, -kp),
                                       __fmaf_rn(fmaxf(d[j + 1], neg_inf()), a.c, -kq));
                beta += ex2_approx(l0);
                b1 += ex2_approx(l1);
            }
        });
        beta = warp_sum(beta + b1);
    }
    if (lane == 0) sh.beta[warp] = beta;
    cluster.sync();
    }
    if (rank == 0 && warp == 0) {
        const int nseg = S * kWarps;
        float b = 0.f;
        for (int s = lane; s < nseg; s += 32) b += cluster.map_shared_rank(&sh, s / kWarps)->beta[s % kWarps];
        b = warp_sum(b);
        if (lane == 0) {
            if (!ok) atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
            const float Lq = log2f(R.Zq), Lp = log2f(R.Zp);
            const float Hq = ok ? fmaxf(kLn2 * (Lq - R.Aq / R.Zq), 0.f) : 0.f;
            const float KL = ok ? fmaxf(kLn2 * (R.D / R.Zq - Lq + Lp), 0.f) : 0.f;
            const float Hqp = Hq + KL;
            float* o = a.out + static_cast<size_t>(r) * 8;
            o[0] = b;
            o[1] = Hq;
            o[2] = Hqp;
            o[3] = KL;
            // gamma = 1 + KL / H_q: where H_q vanishes it is +inf with any divergence and 1 with none
            o[4] = Hq > 0.f ? Hqp / Hq : (KL > 0.f ? __int_as_float(0x7f800000) : 1.0f);
            o[5] = 1.0f - sqrtf(0.5f * KL);
            o[6] = 1.0f - sqrtf(-expm1f(-KL));
            o[7] = 1.0f - sqrtf(a.c_bound * Hq);
        }
    }
    cluster.sync();
}

}  // namespace svip
