// Verification of a tree of draft candidates: several candidates per position, as when the length policy
// runs on top of a tree drafter (Section 3.3).  The paper states no accept rule for that setting; this is the
// published multi-candidate generalisation of Algorithms 2 and 4 (recursive rejection sampling): at a node with
// target distribution p, draft distribution q and candidates x_1..x_m,
//     p_1 = p;   accept x_i if r_i < min(1, p_i(x_i) / q(x_i));   else p_{i+1} = max(0, p_i - q) / S_i,
//     S_i = sum max(0, p_i - q);
// an accepted candidate becomes the current node; when none is accepted (or the node is a leaf) the next token is
// drawn from p_{m+1} (from p at a leaf) and the walk ends.  With one candidate per node it is svip_verify.
//
// One cluster per sequence.  The normalisers of every target row (and draft row) come from row_stats_kernel, as
// in the linear round.  The walk itself is a chain: every thread of the cluster takes the same decisions from the
// same bits (the two logits of the candidate, the normalisers, the masses S_i), and each rejection costs one pass
// over the node's two rows (from L2 after the first one) that sums max(0, p_i - q) per warp segment; the segment
// sums of the last pass are what the inverse CDF of the final draw needs, so the correction costs no further pass.
#pragma once

#include "svip_verify.cuh"

namespace svip {

constexpr int kMaxRejections = 16;   // candidates of one node that can be rejected before the rest is ignored

struct TreeArgs {
    const int32_t* tokens;    // [B, N]
    const int32_t* parent;    // [B, N]: -1 = child of the root, else a lower node index
    const void* q_logits;     // [B, N + 1] rows: root, then the nodes
    long q_row_stride;
    const float2* q_stats;    // per draft row (m, Z)
    const void* t_logits;
    long t_row_stride;
    const float2* p_stats;    // per target row (m, Z)
    int N, V;
    float c;
    const float* uniforms;    // [B, N + 1]: accept draw per node, then the final draw
    int32_t* n_accepted;      // [B]
    int32_t* path;            // [B, N]
    int32_t* next_token;      // [B]
    unsigned* status;
};

// Weights of the distribution after `nrej` rejections at a node, unnormalised: p for nrej == 0, else
// max(0, p_nrej - q) with p_1 = p and p_{i+1} = max(0, p_i - q) * rS[i].
template <int DT>
struct TreeWeights {
    RowGeom gt, gq;
    const void* qrow;
    float c, Mp, rZp, Mq, rZq;
    int nrej;
    float rS[kMaxRejections];   // rS[i] = 1 / S_i, i = 1 .. nrej - 1 (entry 0 unused)
    struct Raw { uint4 t, q; };
    __device__ __forceinline__ float of(float p, float q) const {
        if (nrej == 0) return p;
        float r = p;
        for (int i = 1; i < nrej; ++i) r = fmaxf(r - q, 0.f) * rS[i];
        return fmaxf(r - q, 0.f);
    }
    __device__ __forceinline__ Raw load(int vi) const {
        Raw r;
        r.t = ld_vec(gt.base + vi);
        r.q = (nrej > 0 && gq.pre == gt.pre) ? ld_vec(gq.base + vi) : make_uint4(0, 0, 0, 0);
        return r;
    }
    __device__ __forceinline__ void weights(int vi, const Raw& raw, float (&w)[ElemTraits<DT>::kEPV]) const {
        constexpr int EPV = ElemTraits<DT>::kEPV;
        float x[EPV], d[EPV];
        unpack_masked<DT>(raw.t, vi, gt, x);
        if (nrej > 0) {
            if (gq.pre == gt.pre) {
                unpack_masked<DT>(raw.q, vi, gq, d);
            } else {   // rows with different 16-byte phase: element loads
#pragma unroll
                for (int j = 0; j < EPV; ++j) {
                    int i = vi * EPV + j - gt.pre;
                    d[j] = (i >= 0 && i < gt.V) ? ElemTraits<DT>::load_one(qrow, i) : neg_inf();
                }
            }
        }
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            const float p = ex2_approx(fmaxf(__fmaf_rn(x[j], c, -Mp), kArgFloor)) * rZp;     // NaN / -inf: no mass
            float q = 0.f;
            if (nrej > 0) q = ex2_approx(fmaxf(__fmaf_rn(d[j], c, -Mq), kArgFloor)) * rZq;
            w[j] = of(p, q);
        }
    }
};

struct TreeShared {
    SegPick pick;
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 2) verify_tree_kernel(TreeArgs a) {
    using E = ElemTraits<DT>;
    constexpr int EPV = E::kEPV;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int b = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ SegEntry seg[kWarps];
    __shared__ ScanShared scan;
    __shared__ TreeShared ts;

    pdl_launch_dependents();
    pdl_wait();
    const int N = a.N;
    const int32_t* parent = a.parent + static_cast<size_t>(b) * N;
    const int32_t* tokens = a.tokens + static_cast<size_t>(b) * N;
    const float* un = a.uniforms + static_cast<size_t>(b) * (N + 1);
    int32_t* path = a.path + static_cast<size_t>(b) * N;
    const char* tl = static_cast<const char*>(a.t_logits);
    const char* ql = static_cast<const char*>(a.q_logits);
    const bool writer = rank == 0 && tid == 0;
    if (rank == 0)
        for (int i = tid; i < N; i += kThreads) path[i] = -1;
    __syncthreads();   // the -1 fill is in before thread 0 writes accepted nodes over it

    // Sums the current weights per warp segment, leaves in ts.pick the total and the segment that holds the
    // final draw, identical in every block of the cluster.
    TreeWeights<DT> wf;
    wf.c = a.c;
    const float u_final = un[N];
    auto pass = [&]() {
        int v_lo, v_hi;
        seg_range(wf.gt, rank * kWarps + warp, v_lo, v_hi);
        float acc = 0.f;
        for (int v0 = v_lo + lane; v0 < v_hi; v0 += 128) {
            typename TreeWeights<DT>::Raw raw[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (v0 + 32 * k < v_hi) raw[k] = wf.load(v0 + 32 * k);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (v0 + 32 * k < v_hi) {
                    float w[EPV];
                    wf.weights(v0 + 32 * k, raw[k], w);
#pragma unroll
                    for (int j = 0; j < EPV; ++j) acc += w[j];
                }
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) { seg[warp].m = 0.f; seg[warp].idx = 0; seg[warp].Z = acc; seg[warp].A = 0.f; }
        cluster.sync();
        if (warp == 0) {
            const int nseg = S * kWarps;
            const int per = (nseg + 31) / 32;
            float mass[kSegPerLane];
#pragma unroll
            for (int k = 0; k < kSegPerLane; ++k) {
                const int s = lane * per + k;
                mass[k] = 0.f;
                if (k < per && s < nseg) mass[k] = cluster.map_shared_rank(seg, s / kWarps)[s % kWarps].Z;
            }
            const SegPick p = pick_segment(mass, per, nseg, u_final, lane);
            if (lane == 0) ts.pick = p;
        }
        cluster.sync();   // seg may be rewritten, ts.pick is visible
    };

    int cur = -1, n_acc = 0;
    bool malformed = false;
    for (int step = 0; step <= N; ++step) {
        const long row = static_cast<long>(b) * (N + 1) + cur + 1;
        const char* trow = tl + static_cast<size_t>(row) * a.t_row_stride * E::kBytes;
        const char* qrow = ql + static_cast<size_t>(row) * a.q_row_stride * E::kBytes;
        wf.gt = make_geom<DT>(trow, a.V, S * kWarps);
        wf.gq = make_geom<DT>(qrow, a.V, S * kWarps);
        wf.qrow = qrow;
        const float2 ps = a.p_stats[row];
        wf.Mp = __fmul_rn(ps.x, a.c);
        wf.rZp = 1.0f / ps.y;
        wf.nrej = 0;
        float Zq = 1.f;
        bool have_q = false, pass_valid = false;
        int taken = -1;
        // the children of the current node, in index order
        for (int i = cur + 1; i < N && taken < 0; ++i) {
            const int par = parent[i];
            if (par != cur) {
                if (par < -1 || par >= i) malformed = true;
                continue;
            }
            if (wf.nrej >= kMaxRejections - 1) { malformed = true; break; }
            if (!have_q) {
                const float2 qs = a.q_stats[row];
                Zq = qs.y;
                wf.Mq = __fmul_rn(qs.x, a.c);
                wf.rZq = 1.0f / qs.y;
                have_q = true;
            }
            const int x = tokens[i];
            bool acc = false;
            if (x >= 0 && x < a.V) {
                const float tv = E::load_one(trow, x), dv = E::load_one(qrow, x);
                const bool q_zero = !(dv > neg_inf());
                const float r = un[i];
                if (wf.nrej == 0) {
                    // as in the linear round: the ratio from the difference of the two log2 arguments
                    const float ap = __fmaf_rn(tv, a.c, -wf.Mp);
                    const float aq = __fmaf_rn(dv, a.c, -wf.Mq);
                    const bool p_zero = !(tv > neg_inf());
                    const float d = fminf(fmaxf(ap - aq, -126.f), 126.f);
                    const float num = __fmul_rn(exp2f(d), Zq);
                    acc = !p_zero && (q_zero || num >= ps.y || __fmul_rn(r, ps.y) < num);
                } else {
                    // p_i(x) after the rejections so far; r < p_i / q without the division
                    const float p = ex2_approx(fmaxf(__fmaf_rn(tv, a.c, -wf.Mp), kArgFloor)) * wf.rZp;
                    const float q = q_zero ? 0.f : ex2_approx(fmaxf(__fmaf_rn(dv, a.c, -wf.Mq), kArgFloor)) * wf.rZq;
                    const float pi = wf.of(p, q) * wf.rS[wf.nrej];      // max(0, p_{i-1} - q) / S_{i-1}
                    acc = pi > 0.f && (q_zero || pi >= q || __fmul_rn(r, q) < pi);
                }
            }
            if (acc) { taken = i; break; }
            // rejected: the masses of max(0, p_i - q), whose total is S_i
            wf.nrej += 1;
            pass();
            const float total = ts.pick.total;
            if (total > 0.f) {
                wf.rS[wf.nrej] = 1.0f / total;
                pass_valid = true;
            } else {           // no residual mass (rounding): the distribution stays as it was
                wf.nrej -= 1;
                pass_valid = false;
            }
        }
        if (taken >= 0) {
            if (writer) path[n_acc] = taken;
            ++n_acc;
            cur = taken;
            continue;
        }
        // no candidate accepted (or a leaf): the next token from the current distribution
        if (!pass_valid) pass();
        const SegPick P = ts.pick;
        int token = 0;
        if (P.total > 0.f) {
            if (P.seg / kWarps == rank) {
                int v_lo, v_hi;
                seg_range(wf.gt, P.seg, v_lo, v_hi);
                const int virt = fine_scan<EPV>(wf, v_lo, v_hi, P.prefix, P.target, scan, tid, lane, warp);
                token = virt >= 0 ? virt - wf.gt.pre : 0;
                if (tid == 0) a.next_token[b] = token;
            }
        } else if (writer) {
            atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
            a.next_token[b] = 0;
        }
        break;
    }
    if (writer) {
        a.n_accepted[b] = n_acc;
        if (malformed) atomicOr(a.status, SVIP_STATUS_BAD_TREE);
    }
}

// Greedy: a child is accepted iff its token is the argmax of the node's target row (Algorithm 3 at every
// node); otherwise that argmax is the next token (Algorithm 5).  One thread per sequence.
struct TreeGreedyArgs {
    const int32_t* tokens;
    const int32_t* parent;
    const int32_t* p_argmax;   // per target row
    int B, N;
    int32_t* n_accepted;
    int32_t* path;
    int32_t* next_token;
};

__global__ void __launch_bounds__(kPolicyThreads) verify_tree_greedy_kernel(TreeGreedyArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * kPolicyThreads + threadIdx.x;
    if (b >= a.B) return;
    const int N = a.N;
    const int32_t* parent = a.parent + static_cast<size_t>(b) * N;
    const int32_t* tokens = a.tokens + static_cast<size_t>(b) * N;
    int32_t* path = a.path + static_cast<size_t>(b) * N;
    for (int i = 0; i < N; ++i) path[i] = -1;
    int cur = -1, n = 0;
    for (int step = 0; step <= N; ++step) {
        const int am = a.p_argmax[static_cast<size_t>(b) * (N + 1) + cur + 1];
        int taken = -1;
        for (int i = cur + 1; i < N && taken < 0; ++i)
            if (parent[i] == cur && tokens[i] == am) taken = i;
        if (taken < 0) { a.next_token[b] = am; break; }
        path[n++] = taken;
        cur = taken;
    }
    a.n_accepted[b] = n;
}

}  // namespace svip
