// The analysis quantities of a (target row, draft row) pair (Eq. 1-6, appendix B).
#pragma once

#include "svip_draft.cuh"

namespace svip {
// ------------------------------------------------------------------ analysis quantities of a row pair
//
// Eq. 1-6 and appendix B: for p = softmax(target row / T) and q = softmax(draft row / T), with the
// normalisers already known, one pass over both rows accumulates
//   beta = sum min(p, q),   sum q * log2 q,   sum q * (log2 q - log2 p)
// from which H_q, KL(q||p), the cross entropy H_qp = H_q + KL, gamma = H_qp / H_q and the three lower
// bounds on beta follow.  KL is accumulated directly (not as a difference of two entropies) so that
// it keeps its relative precision when p is close to q.

struct PairArgs {
    const void* t_logits;
    long t_row_stride;
    const void* q_logits;
    long q_row_stride;
    const float2* p_stats;
    const float2* q_stats;
    int V;
    float c;
    float c_bound;
    float* out;   // [pairs][8]
    unsigned* status;
};

struct PairSums {
    float beta, qlq, kl;
};

template <int DT>
__global__ void __launch_bounds__(kThreads) pair_stats_kernel(PairArgs a) {
    using E = ElemTraits<DT>;
    constexpr int EPV = E::kEPV;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int r = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ PairSums part[kWarps];

    pdl_launch_dependents();
    const char* trow = static_cast<const char*>(a.t_logits) + static_cast<size_t>(r) * a.t_row_stride * E::kBytes;
    const char* qrow = static_cast<const char*>(a.q_logits) + static_cast<size_t>(r) * a.q_row_stride * E::kBytes;
    const RowGeom gt = make_geom<DT>(trow, a.V, S * kWarps);
    const RowGeom gq = make_geom<DT>(qrow, a.V, S * kWarps);
    pdl_wait();
    const float2 ps = a.p_stats[r], qs = a.q_stats[r];
    const float Mp = __fmul_rn(ps.x, a.c), Mq = __fmul_rn(qs.x, a.c);
    const float Lp = log2f(ps.y), Lq = log2f(qs.y);
    const float rZp = 1.0f / ps.y, rZq = 1.0f / qs.y;
    int v_lo, v_hi;
    seg_range(gt, rank * kWarps + warp, v_lo, v_hi);
    float beta = 0.f, qlq = 0.f, kl = 0.f;
#pragma unroll 2
    for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
        float x[EPV], d[EPV];
        unpack_masked<DT>(__ldg(gt.base + vi), vi, gt, x);
        if (gq.pre == gt.pre) {
            unpack_masked<DT>(__ldg(gq.base + vi), vi, gq, d);
        } else {
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                int i = vi * EPV + j - gt.pre;
                d[j] = (i >= 0 && i < gt.V) ? E::load_one(qrow, i) : neg_inf();
            }
        }
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            float ap = __fmaf_rn(x[j], a.c, -Mp);      // log2 of the unnormalised p
            float aq = __fmaf_rn(d[j], a.c, -Mq);
            if (!(ap == ap)) ap = neg_inf();            // NaN logits count as masked
            float p = ex2_approx(fmaxf(ap, kArgFloor)) * rZp;
            float q = ex2_approx(fmaxf(aq, kArgFloor)) * rZq;   // NaN -> floor -> 0
            beta += fminf(p, q);
            if (q > 0.f) {
                float lq = aq - Lq;
                qlq = __fmaf_rn(q, lq, qlq);
                kl = __fmaf_rn(q, lq - (ap - Lp), kl);   // +inf where p is masked but q is not
            }
        }
    }
    beta = warp_sum(beta); qlq = warp_sum(qlq); kl = warp_sum(kl);
    if (lane == 0) { part[warp].beta = beta; part[warp].qlq = qlq; part[warp].kl = kl; }
    cluster.sync();
    if (rank == 0 && warp == 0) {
        const int nseg = S * kWarps;
        float b = 0.f, s1 = 0.f, s3 = 0.f;
        for (int s = lane; s < nseg; s += 32) {
            const PairSums v = cluster.map_shared_rank(part, s / kWarps)[s % kWarps];
            b += v.beta; s1 += v.qlq; s3 += v.kl;
        }
        b = warp_sum(b); s1 = warp_sum(s1); s3 = warp_sum(s3);
        if (lane == 0) {
            const bool ok = ps.y > 0.f && qs.y > 0.f && fabsf(ps.x) <= kMaxLogit && fabsf(qs.x) <= kMaxLogit;
            if (!ok) atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
            const float Hq = fmaxf(-kLn2 * s1, 0.f);
            const float KL = fmaxf(kLn2 * s3, 0.f);
            const float Hqp = Hq + KL;
            float* o = a.out + static_cast<size_t>(r) * 8;
            o[0] = b;
            o[1] = Hq;
            o[2] = Hqp;
            o[3] = KL;
            o[4] = Hqp / Hq;
            o[5] = 1.0f - sqrtf(0.5f * KL);
            o[6] = 1.0f - sqrtf(-expm1f(-KL));
            o[7] = 1.0f - sqrtf(a.c_bound * Hq);
        }
    }
    cluster.sync();
}

}  // namespace svip
