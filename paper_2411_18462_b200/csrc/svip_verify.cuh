// Target side: accept test, first rejection, correction / bonus token (Algorithms 2-5; Algorithm 1 outer-loop body).
#pragma once

#include "svip_draft.cuh"

namespace svip {
// ------------------------------------------------------------------ verify, phase 2 (sampling)

struct FinishArgs {
    const int32_t* draft_tokens;
    const void* q_logits;
    long q_row_stride;
    const float2* q_stats_user;   // indexed by draft row, or NULL
    const float2* q_stats_ws;     // indexed by target row (used when q_stats_user is NULL)
    long q_seq_stride, q_pos_stride;
    const void* t_logits;
    long t_row_stride;
    const float2* p_stats;        // indexed by target row
    const int32_t* cu;
    int K, V;
    float c;
    const float* uniforms;
    int32_t* n_accepted;
    int32_t* next_token;
    unsigned* status;
    const float* p_thr;           // kThr: truncation threshold of every target row
    const float* q_thr;           // kThr: ... of every draft row (indexed like the draft tokens)
    const int32_t* n_acc_in;      // not NULL: the first rejection of every sequence is already known
    float2* p_stats_out;          // verify_scan_kernel: (max, Z) of every target row it read, by target row
};

// Weights max(0, p - q) of Algorithm 4 (or p alone for the bonus token) for one vector.
template <int DT>
struct ResidualWeights {
    RowGeom gt, gq;
    const void* qrow;
    float c, Mp, rZp, Mq, rZq;
    int bonus;
    float thr_p = -INFINITY, thr_q = -INFINITY;   // truncated distributions: logits below carry nothing
    struct Raw { uint4 t, q; };
    __device__ __forceinline__ Raw load(int vi) const {
        Raw r;
        r.t = ld_vec(gt.base + vi);
        r.q = (!bonus && gq.pre == gt.pre) ? ld_vec(gq.base + vi) : make_uint4(0, 0, 0, 0);
        return r;
    }
    __device__ __forceinline__ void operator()(int vi, float (&w)[ElemTraits<DT>::kEPV]) const {
        weights(vi, load(vi), w);
    }
    __device__ __forceinline__ void weights(int vi, const Raw& raw, float (&w)[ElemTraits<DT>::kEPV]) const {
        constexpr int EPV = ElemTraits<DT>::kEPV;
        float x[EPV];
        unpack_masked<DT>(raw.t, vi, gt, x);
#pragma unroll
        for (int j = 0; j < EPV; ++j)
            w[j] = x[j] >= thr_p ? ex2_approx(fmaxf(__fmaf_rn(x[j], c, -Mp), kArgFloor)) * rZp : 0.f;
        if (bonus) return;
        float d[EPV];
        if (gq.pre == gt.pre) {
            unpack_masked<DT>(raw.q, vi, gq, d);
        } else {
            // rows with different 16-byte phase: element loads
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                int i = vi * EPV + j - gt.pre;
                d[j] = (i >= 0 && i < gt.V) ? ElemTraits<DT>::load_one(qrow, i) : neg_inf();
            }
        }
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            float q = d[j] >= thr_q ? ex2_approx(fmaxf(__fmaf_rn(d[j], c, -Mq), kArgFloor)) * rZq : 0.f;
            w[j] = fmaxf(w[j] - q, 0.f);
        }
    }
};

// Sum of the residual (or bonus) weights over one warp segment, streamed through the cp.async ring:
// four stages for the target row and four for the draft row.  Same arithmetic as
// ResidualWeights::weights (packed), without its masking: vectors that stick out of the row, and
// rows whose draft row has another 16-byte phase, go through the functor instead.
template <int DT, bool kThr>
__device__ __forceinline__ float residual_segment_sum(const ResidualWeights<DT>& wf, int seg, int lane,
                                                      uint32_t slot0) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    constexpr uint32_t kSlotStride = kThreads * 16;
    constexpr int kDepth = kStages / 2;
    const RowGeom& g = wf.gt;
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    float acc = 0.f;
    if (!wf.bonus && wf.gq.pre != g.pre) {
        for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
            float w[EPV];
            wf(vi, w);
#pragma unroll
            for (int j = 0; j < EPV; ++j) acc += w[j];
        }
        return acc;
    }
    const bool head_edge = g.pre > 0;
    const bool tail_edge = ((g.pre + g.V) % EPV) != 0;
    int i_lo = v_lo, i_hi = v_hi;
    if (head_edge && v_lo == 0 && v_hi > 0) i_lo = 1;
    if (tail_edge && v_hi == g.nvec && i_hi > i_lo) i_hi = g.nvec - 1;
    const int vi0 = i_lo + lane;
    const int n = i_hi > vi0 ? (i_hi - vi0 + 31) >> 5 : 0;
    const uint4* st = g.base + vi0;
    const uint4* sq = wf.gq.base + vi0;
    const bool two = !wf.bonus;
#pragma unroll
    for (int s = 0; s < kDepth; ++s) {
        if (s < n) {
            cp_async16(slot0 + s * kSlotStride, st + 32 * s);
            if (two) cp_async16(slot0 + (kDepth + s) * kSlotStride, sq + 32 * s);
        }
        cp_async_commit();
    }
    const f32x2 c2 = pack2(wf.c, wf.c);
    const f32x2 nmp2 = pack2(-wf.Mp, -wf.Mp), nmq2 = pack2(-wf.Mq, -wf.Mq);
    const f32x2 rzp2 = pack2(wf.rZp, wf.rZp), rzq2 = pack2(wf.rZq, wf.rZq);
    float acc1 = 0.f;
    for (int it = 0; it < n; ++it) {
        cp_async_wait<kDepth - 1>();
        const uint32_t sa = slot0 + (it & (kDepth - 1)) * kSlotStride;
        const uint4 rt = lds128(sa);
        uint4 rq = make_uint4(0, 0, 0, 0);
        if (two) rq = lds128(sa + kDepth * kSlotStride);
        const int nx = it + kDepth;
        if (nx < n) {
            cp_async16(sa, st + 32 * nx);
            if (two) cp_async16(sa + kDepth * kSlotStride, sq + 32 * nx);
        }
        cp_async_commit();
        float x[EPV], d[EPV];
        ElemTraits<DT>::unpack(rt, x);
        ElemTraits<DT>::unpack(rq, d);
        if (kThr) {
            drop_below<EPV>(x, wf.thr_p);
            drop_below<EPV>(d, wf.thr_q);
        }
#pragma unroll
        for (int j = 0; j < EPV; j += 2) {
            float a0, a1;
            unpack2(fma2(pack2(x[j], x[j + 1]), c2, nmp2), a0, a1);
            f32x2 p2 = mul2(pack2(ex2_approx(a0), ex2_approx(a1)), rzp2);
            float p0, p1;
            unpack2(p2, p0, p1);
            if (two) {
                unpack2(fma2(pack2(d[j], d[j + 1]), c2, nmq2), a0, a1);
                f32x2 q2 = mul2(pack2(ex2_approx(a0), ex2_approx(a1)), rzq2);
                float q0, q1;
                unpack2(q2, q0, q1);
                p0 = fmaxf(p0 - q0, 0.f);
                p1 = fmaxf(p1 - q1, 0.f);
            }
            acc += p0;
            acc1 += p1;
        }
    }
    cp_async_wait<0>();
    acc += acc1;
    if (lane == 0) {
        float w[EPV];
        if (head_edge && v_lo == 0 && v_hi > 0) {
            wf(0, w);
#pragma unroll
            for (int j = 0; j < EPV; ++j) acc += w[j];
        }
        if (tail_edge && v_hi == g.nvec && v_lo < v_hi && !(g.nvec == 1 && head_edge)) {
            wf(g.nvec - 1, w);
#pragma unroll
            for (int j = 0; j < EPV; ++j) acc += w[j];
        }
    }
    // NaN weights (NaN logits) count as zero in the functor; here they would poison the sum
    if (!(acc == acc)) {
        acc = 0.f;
        for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
            float w[EPV];
            wf(vi, w);
#pragma unroll
            for (int j = 0; j < EPV; ++j) acc += w[j];
        }
    }
    return acc;
}

// Algorithm 2 for one position: r < min(1, p(x)/q(x)), from the two logits of the drafted token and the
// (max, Z) of the two rows.  p(x)/q(x) = 2^(ap - aq) * Zq / Zp, from the difference of the two log2
// arguments, so that a token however unlikely under both models keeps its ratio (no underflow).  No
// division: a ratio >= 1 accepts every r in [0,1); p(x) == 0 accepts none; q(x) == 0 < p(x) is a ratio of
// +inf.  `p_out` / `q_out`: the token lies outside the truncated support of that side.
__device__ __forceinline__ bool accept_test(float tv, float dv, float2 ps, float2 qs, float c, float r,
                                            bool p_out, bool q_out) {
    const float ap = __fmaf_rn(tv, c, -__fmul_rn(ps.x, c));
    const float aq = __fmaf_rn(dv, c, -__fmul_rn(qs.x, c));
    const bool p_zero = p_out || !(tv > neg_inf());   // NaN counts as -inf
    const bool q_zero = q_out || !(dv > neg_inf());
    const float d = fminf(fmaxf(ap - aq, -126.f), 126.f);
    const float num = __fmul_rn(exp2f(d), qs.y);
    return !p_zero && (q_zero || num >= ps.y || __fmul_rn(r, ps.y) < num);
}

struct FinishShared {
    int n_acc;
    SegPick pick;
};

// Correction token from max(0, p - q) of the first rejected position, or bonus token from p of the row after
// the last draft token (Algorithms 4 and 5), for sequence i whose number of accepted tokens is known.  Run by
// every thread of the sequence's cluster; writes n_accepted[i] and next_token[i].
template <int DT, bool kThr>
__device__ __forceinline__ void finish_sequence(const FinishArgs& a, cg::cluster_group& cluster, int S, int rank,
                                                int i, int row0, int Ki, long dbase, long dstep, int n_acc,
                                                float2 ps, SegEntry* seg, ScanShared& scan, FinishShared& fs,
                                                uint32_t slot0) {
    using E = ElemTraits<DT>;
    constexpr int EPV = E::kEPV;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const char* tl = static_cast<const char*>(a.t_logits);
    const char* ql = static_cast<const char*>(a.q_logits);
    const float u = a.uniforms[row0 + Ki];

    ResidualWeights<DT> wf;
    const char* trow = tl + static_cast<size_t>(row0 + n_acc) * a.t_row_stride * E::kBytes;
    wf.gt = make_geom<DT>(trow, a.V, S * kWarps);
    wf.c = a.c;
    wf.Mp = __fmul_rn(ps.x, a.c);
    wf.rZp = 1.0f / ps.y;
    if (kThr) wf.thr_p = a.p_thr[row0 + n_acc];
    wf.bonus = n_acc >= Ki;
    wf.qrow = nullptr; wf.gq = wf.gt; wf.Mq = 0.f; wf.rZq = 0.f;
    if (!wf.bonus) {
        long dr = dbase + n_acc * dstep;
        wf.qrow = ql + static_cast<size_t>(dr) * a.q_row_stride * E::kBytes;
        wf.gq = make_geom<DT>(wf.qrow, a.V, S * kWarps);
        float2 qs = a.q_stats_user ? a.q_stats_user[dr] : a.q_stats_ws[row0 + n_acc];
        wf.Mq = __fmul_rn(qs.x, a.c);
        wf.rZq = 1.0f / qs.y;
        if (kThr) wf.thr_q = a.q_thr[dr];
    }

    int token = -1;
    for (int pass = 0; pass < 2; ++pass) {
        // mass of this warp's segment
        int v_lo, v_hi;
        float acc = residual_segment_sum<DT, kThr>(wf, rank * kWarps + warp, lane, slot0);
        acc = warp_sum(acc);
        if (lane == 0) { seg[warp].m = 0.f; seg[warp].idx = 0; seg[warp].Z = acc; seg[warp].A = 0.f; }
        cluster.sync();
        if (warp == 0) {
            const int nseg = S * kWarps;
            const int per = (nseg + 31) / 32;
            float mass[kSegPerLane];
#pragma unroll
            for (int k = 0; k < kSegPerLane; ++k) {
                int s = lane * per + k;
                mass[k] = 0.f;
                if (k < per && s < nseg) mass[k] = cluster.map_shared_rank(seg, s / kWarps)[s % kWarps].Z;
            }
            SegPick p = pick_segment(mass, per, nseg, u, lane);
            if (lane == 0) fs.pick = p;
        }
        cluster.sync();
        const SegPick P = fs.pick;
        if (P.total > 0.f) {
            if (P.seg / kWarps == rank) {
                seg_range(wf.gt, P.seg, v_lo, v_hi);
                int virt = fine_scan<EPV>(wf, v_lo, v_hi, P.prefix, P.target, scan, tid, lane, warp);
                token = virt >= 0 ? virt - wf.gt.pre : 0;
            }
            break;
        }
        // No residual mass (p == q wherever it matters): fall back to sampling from p.
        if (wf.bonus) {
            if (rank == 0 && tid == 0) atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
            if (rank == 0) token = 0;
            break;
        }
        wf.bonus = 1;
    }
    if (tid == 0) {
        if (rank == 0) a.n_accepted[i] = n_acc;
        if (token >= 0) a.next_token[i] = token;
    }
}

template <int DT, bool kThr = false>
__global__ void __launch_bounds__(kThreads, 2) verify_finish_kernel(FinishArgs a) {
    using E = ElemTraits<DT>;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int i = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ SegEntry seg[kWarps];
    __shared__ ScanShared scan;
    __shared__ FinishShared fs;
    extern __shared__ uint4 ring[];
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;

    pdl_launch_dependents();
    pdl_wait();
    const int row0 = a.cu ? a.cu[i] : i * (a.K + 1);
    const int Ki = a.cu ? a.cu[i + 1] - row0 - 1 : a.K;
    const long dbase = a.q_seq_stride < 0 ? static_cast<long>(row0 - i) : i * a.q_seq_stride;
    const long dstep = a.q_seq_stride < 0 ? 1 : a.q_pos_stride;
    const char* tl = static_cast<const char*>(a.t_logits);
    const char* ql = static_cast<const char*>(a.q_logits);

    // Algorithm 2 at every position at once; the first rejection is the lowest set bit.
    if (a.n_acc_in) {
        if (tid == 0) fs.n_acc = min(max(a.n_acc_in[i], 0), Ki);
    } else if (warp == 0) {
        int n_acc = Ki;
        for (int j0 = 0; j0 < Ki; j0 += 32) {
            int j = j0 + lane;
            bool rej = false;
            if (j < Ki) {
                long dr = dbase + j * dstep;
                int x = a.draft_tokens[dr];
                bool acc = false;
                if (x >= 0 && x < a.V) {
                    float tv = E::load_one(tl + static_cast<size_t>(row0 + j) * a.t_row_stride * E::kBytes, x);
                    float dv = E::load_one(ql + static_cast<size_t>(dr) * a.q_row_stride * E::kBytes, x);
                    float2 ps = a.p_stats[row0 + j];
                    float2 qs = a.q_stats_user ? a.q_stats_user[dr] : a.q_stats_ws[row0 + j];
                    bool p_out = false, q_out = false;
                    if (kThr) {   // tokens that the truncation dropped have probability zero
                        p_out = !(tv >= a.p_thr[row0 + j]);
                        q_out = !(dv >= a.q_thr[dr]);
                    }
                    acc = accept_test(tv, dv, ps, qs, a.c, a.uniforms[row0 + j], p_out, q_out);
                }
                rej = !acc;
            }
            unsigned mask = __ballot_sync(0xffffffffu, rej);
            if (mask) { n_acc = j0 + __ffs(mask) - 1; break; }
        }
        if (lane == 0) fs.n_acc = n_acc;
    }
    __syncthreads();
    const int n_acc = fs.n_acc;
    finish_sequence<DT, kThr>(a, cluster, S, rank, i, row0, Ki, dbase, dstep, n_acc, a.p_stats[row0 + n_acc], seg,
                              scan, fs, slot0);
}

// ------------------------------------------------------------------ verify, phase 2 (greedy)

struct GreedyArgs {
    const int32_t* draft_tokens;
    const int32_t* p_argmax;
    const int32_t* cu;
    long q_seq_stride, q_pos_stride;
    int B, K;
    int32_t* n_accepted;
    int32_t* next_token;
};

__global__ void __launch_bounds__(kThreads) verify_greedy_kernel(GreedyArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (i >= a.B) return;
    const int row0 = a.cu ? a.cu[i] : i * (a.K + 1);
    const int Ki = a.cu ? a.cu[i + 1] - row0 - 1 : a.K;
    const long dbase = a.q_seq_stride < 0 ? static_cast<long>(row0 - i) : i * a.q_seq_stride;
    const long dstep = a.q_seq_stride < 0 ? 1 : a.q_pos_stride;
    int n_acc = Ki;
    for (int j0 = 0; j0 < Ki; j0 += 32) {
        int j = j0 + lane;
        bool rej = false;
        if (j < Ki) rej = a.draft_tokens[dbase + j * dstep] != a.p_argmax[row0 + j];
        unsigned mask = __ballot_sync(0xffffffffu, rej);
        if (mask) { n_acc = j0 + __ffs(mask) - 1; break; }
    }
    if (lane == 0) {
        a.n_accepted[i] = n_acc;
        a.next_token[i] = a.p_argmax[row0 + n_acc];
    }
}

// ------------------------------------------------------------------ verify with early exit

struct WalkShared {
    // what the accept test of positions j0 .. j0+31 needs besides the target row's statistics
    float tv[32], dv[32], r[32];
    float2 qs[32];
    int x[32];
    int go;                       // decision of the current row: 1 = accepted, read the next row
    float2 ps;                    // (max, Z) of the current row
};

// The accept tests of a sequence stop at its first rejection (Algorithm 1, verify loop), so the target rows
// after it are never needed.  One cluster per sequence reads the target rows in order: statistics of row j,
// accept test of position j (Algorithm 2 / 3), next row only if accepted; then the correction or bonus token
// from the row it stopped at (Algorithms 4 and 5).  Also writes the (max, Z) of every row it read.
template <int DT, bool kGreedy>
__global__ void __launch_bounds__(kThreads, 2) verify_scan_kernel(FinishArgs a) {
    using E = ElemTraits<DT>;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int i = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ SegEntry seg[2][kWarps];   // by row parity: a peer may still read row j while row j+1 is reduced
    __shared__ WalkShared sh;
    __shared__ ScanShared scan;
    __shared__ FinishShared fs;
    extern __shared__ uint4 ring[];
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;

    pdl_launch_dependents();
    pdl_wait();
    const int row0 = a.cu ? a.cu[i] : i * (a.K + 1);
    const int Ki = a.cu ? a.cu[i + 1] - row0 - 1 : a.K;
    const long dbase = a.q_seq_stride < 0 ? static_cast<long>(row0 - i) : i * a.q_seq_stride;
    const long dstep = a.q_seq_stride < 0 ? 1 : a.q_pos_stride;
    const char* tl = static_cast<const char*>(a.t_logits);
    const char* ql = static_cast<const char*>(a.q_logits);

    int n_acc = Ki;
    int last_idx = 0;
    for (int j = 0; j <= Ki; ++j) {
        if ((j & 31) == 0 && j < Ki) {
            // the drafted tokens of the next 32 positions, their two logits, the draft rows' statistics
            __syncthreads();
            if (warp == 0 && j + lane < Ki) {
                const int jj = j + lane;
                const long dr = dbase + jj * dstep;
                const int x = a.draft_tokens[dr];
                sh.x[lane] = x;
                if (!kGreedy) {
                    const bool in = x >= 0 && x < a.V;
                    sh.tv[lane] = in ? E::load_one(tl + static_cast<size_t>(row0 + jj) * a.t_row_stride * E::kBytes, x) : 0.f;
                    sh.dv[lane] = in ? E::load_one(ql + static_cast<size_t>(dr) * a.q_row_stride * E::kBytes, x) : 0.f;
                    sh.qs[lane] = a.q_stats_user ? a.q_stats_user[dr] : a.q_stats_ws[row0 + jj];
                    sh.r[lane] = a.uniforms[row0 + jj];
                }
            }
        }
        const char* trow = tl + static_cast<size_t>(row0 + j) * a.t_row_stride * E::kBytes;
        const RowGeom g = make_geom<DT>(trow, a.V, S * kWarps);
        SegEntry* mine = seg[j & 1];
        Partial t = reduce_segment<DT, kGreedy ? 0 : 1, kGreedy, false>(g, rank * kWarps + warp, a.c, lane, slot0, neg_inf());
        if (lane == 0) { mine[warp].m = t.m; mine[warp].idx = t.idx; mine[warp].Z = t.Z; mine[warp].A = t.A; }
        cluster.sync();
        if (warp == 0) {
            Partial r; SegPick p;
            combine_segments<kGreedy ? 0 : 1>(cluster, mine, S, a.c, 0.f, lane, r, p);
            const bool ok = fabsf(r.m) <= kMaxLogit && (kGreedy || r.Z > 0.f);
            const int idx = (r.idx >= 0 && r.idx < a.V) ? r.idx : 0;
            int go = 0;
            if (j < Ki) {
                const int k = j & 31;
                const int x = sh.x[k];
                if (kGreedy) go = x == idx;
                else if (x >= 0 && x < a.V)
                    go = accept_test(sh.tv[k], sh.dv[k], make_float2(r.m, r.Z), sh.qs[k], a.c, sh.r[k], false, false);
            }
            if (lane == 0) {
                sh.go = go;
                sh.ps = make_float2(r.m, r.Z);
                if (rank == 0) {
                    if (!ok) atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
                    if (!kGreedy) a.p_stats_out[row0 + j] = make_float2(r.m, r.Z);
                }
            }
            last_idx = idx;
        }
        __syncthreads();
        if (!sh.go) { n_acc = j; break; }
    }
    if (kGreedy) {
        if (rank == 0 && tid == 0) { a.n_accepted[i] = n_acc; a.next_token[i] = last_idx; }
        cluster.sync();   // no block leaves while a peer may still read its segment entries
    } else {
        // the entries of row n_acc - 1 have been read by every peer (they passed the barrier of row n_acc)
        finish_sequence<DT, false>(a, cluster, S, rank, i, row0, Ki, dbase, dstep, n_acc, sh.ps, seg[(n_acc + 1) & 1],
                                   scan, fs, slot0);
    }
}

}  // namespace svip
