// SVIP speculative-decoding epilogues for sm_100a: kernels and the C ABI (see include/svip.h).
//
// Kernels
//   draft_step_kernel    Algorithm 1 inner loop + Eq. 7: one pass over a logits row gives
//                        max / mass / entropy term / argmax; the sampled token is then found by
//                        re-reading one warp segment.  A row is shared by a thread-block
//                        cluster (1..8 blocks) whose partials meet in distributed shared memory.
//   row_stats_kernel     softmax normalisers (or argmax, greedy) of target rows, and of draft
//                        rows when the caller has no q_stats.
//   verify_finish_kernel Algorithms 2 and 4 + the loop of Algorithm 1: ratio tests by one warp
//                        (ballot + first set bit = first rejection), then the residual
//                        max(0, p - q) or the bonus row is sampled by inverse CDF.
//   verify_greedy_kernel Algorithms 3 and 5 on the per-row argmax.
//   pack_ragged_kernel   exclusive scan of (K_i + 1) and the row -> (sequence, position) maps.
#include "svip_device.cuh"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <new>

#include "svip.h"

namespace svip {

constexpr int kPolicyThreads = 256;

struct SegEntry {
    float m;
    int idx;
    float Z;
    float A;
};

// Reads every segment entry of the cluster (warp-collective, run by warp 0 of each block), merges
// them into the row's partial and selects the segment holding the mass u * Z.
template <int kMode>
__device__ __forceinline__ void combine_segments(cg::cluster_group& cluster, SegEntry* seg, int S,
                                                 float c, float u, int lane, Partial& row,
                                                 SegPick& pick, float abs_target = -1.f) {
    const int nseg = S * kWarps;
    const int per = (nseg + 31) / 32;
    Partial e[kSegPerLane];
    float m = neg_inf();
#pragma unroll
    for (int k = 0; k < kSegPerLane; ++k) {
        e[k].m = neg_inf(); e[k].idx = kIntMax; e[k].Z = 0.f; e[k].A = 0.f;
        int s = lane * per + k;
        if (k < per && s < nseg) {
            const SegEntry* remote = cluster.map_shared_rank(seg, s / kWarps);
            SegEntry v = remote[s % kWarps];
            e[k].m = v.m; e[k].idx = v.idx; e[k].Z = v.Z; e[k].A = v.A;
        }
        m = fmaxf(m, e[k].m);
    }
    m = warp_max(m);
    int idx = kIntMax;
    float mass[kSegPerLane];
    float asum = 0.f;
#pragma unroll
    for (int k = 0; k < kSegPerLane; ++k) {
        if (e[k].m == m) idx = min(idx, e[k].idx);
        rescale_to<kMode>(e[k], m, c);
        mass[k] = e[k].Z;
        asum += e[k].A;
    }
    row.m = m;
    row.idx = warp_min_int(idx);
    row.A = warp_sum(asum);
    pick = pick_segment(mass, per, nseg, u, lane, abs_target);
    row.Z = pick.total;
}

// Fine scan of one segment by the whole block.  `wf(vi, w)` yields the weights of the elements
// of vector vi.  Each thread sums a run of consecutive vectors, one block scan places the runs,
// and the thread whose run crosses `target` walks its run again element by element.  Returns the
// virtual element index (vector * EPV + element) of the first element whose cumulative weight
// exceeds `target`, else the last element with positive weight, else -1.
template <int EPV, class WF>
__device__ __forceinline__ int fine_scan(WF& wf, int v_lo, int v_hi, float prefix, float target,
                                         ScanShared& sh, int tid, int lane, int warp) {
    constexpr int kRun = 4;
    const int nv = v_hi - v_lo;
    const int run = min(kRun, max(1, (nv + kThreads - 1) / kThreads));
    if (tid == 0) { sh.hit = kIntMax; sh.lastpos = -1; sh.result = -1; }
    float running = prefix;
    for (int cb = v_lo; cb < v_hi; cb += kThreads * run) {
        const int first = cb + tid * run;
        float ls = 0.f;
        int lastv = -1;
        for (int k = 0; k < run; ++k) {
            int vi = first + k;
            if (vi < v_hi) {
                float w[EPV];
                wf(vi, w);
                float sv = 0.f;
#pragma unroll
                for (int j = 0; j < EPV; ++j) sv += w[j];
                if (sv > 0.f) lastv = vi;
                ls += sv;
            }
        }
        float total;
        const float lo = running + block_scan_excl(ls, sh.wsum, lane, warp, total);
        if (ls > 0.f && lo + ls > target) atomicMin(&sh.hit, tid);
        if (lastv >= 0) atomicMax(&sh.lastpos, lastv);
        __syncthreads();
        const int win = sh.hit;
        if (win != kIntMax) {
            if (tid == win) {
                float cum = lo;
                int res = -1, last = -1;
                for (int k = 0; k < run; ++k) {
                    int vi = first + k;
                    if (vi < v_hi) {
                        float w[EPV];
                        wf(vi, w);
#pragma unroll
                        for (int j = 0; j < EPV; ++j) {
                            cum += w[j];
                            if (w[j] > 0.f) {
                                last = vi * EPV + j;
                                if (cum > target && res < 0) res = last;
                            }
                        }
                    }
                }
                sh.result = res >= 0 ? res : last;
            }
            __syncthreads();
            return sh.result;
        }
        running += total;
    }
    // rounding left nothing above the target: the last element with weight
    const int lv = sh.lastpos;
    if (lv < 0) return -1;
    if (tid == 0) {
        float w[EPV];
        wf(lv, w);
        int last = -1;
#pragma unroll
        for (int j = 0; j < EPV; ++j)
            if (w[j] > 0.f) last = lv * EPV + j;
        sh.result = last;
    }
    __syncthreads();
    return sh.result;
}

// ------------------------------------------------------------------ draft step

struct DraftArgs {
    const void* logits;
    long row_stride;
    int V;
    float c;          // log2(e) / T   (T = 1 when greedy)
    float thresh;
    int greedy;
    const float* uniforms;
    int32_t* token;
    float* entropy;
    uint8_t* stop;
    float* row_stats;
    unsigned* status;
    const uint8_t* active;   // NULL, or one flag per row: rows with 0 are skipped
    const float* ext_target; // NULL, or per row the mass to find (units of this row's own Z), see svip_vp_locate
    int token_offset;        // added to the sampled index (vocabulary shard offset)
    const int32_t* pos;      // NULL, or per row the draft position p whose logits are read (svip_draft_step_at)
    long pos_stride;         // elements between the logits of consecutive positions of a row
    long slot_stride;        // uniforms / token / entropy / row_stats live at index p * slot_stride + row
    const float* thr;        // NULL, or per row the truncation threshold: only logits >= thr[row] count
};

template <int DT>
struct SoftmaxWeights {
    RowGeom g;
    float c, M;
    float thr = -INFINITY;   // logits below it carry no weight (truncated distributions)
    __device__ __forceinline__ void operator()(int vi, float (&w)[ElemTraits<DT>::kEPV]) const {
        constexpr int EPV = ElemTraits<DT>::kEPV;
        float x[EPV];
        unpack_masked<DT>(g.base[vi], vi, g, x);
#pragma unroll
        for (int j = 0; j < EPV; ++j)
            w[j] = x[j] >= thr ? ex2_approx(fmaxf(__fmaf_rn(x[j], c, -M), kArgFloor)) : 0.f;
    }
};

struct RowShared {
    Partial row;
    SegPick pick;
};

// kBlocks is the number of blocks the register budget must leave room for on one SM: 2 for
// launches that fit the GPU in one wave (latency matters, registers are free), 3 for launches of
// many waves, where a third resident block streams on while another one is in its epilogue.
// kPos compiles the position-indexed form (svip_draft_step_at) in, kThr the truncated form
// (svip_draft_step_filtered).
template <int DT, bool kGreedy, int kBlocks, bool kPos = false, bool kThr = false>
__global__ void __launch_bounds__(kThreads, kBlocks) draft_step_kernel(DraftArgs a) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    extern __shared__ uint4 ring[];
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int row = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ SegEntry seg[kWarps];
    __shared__ ScanShared scan;
    __shared__ RowShared res;

    pdl_launch_dependents();
    const char* rp = static_cast<const char*>(a.logits) +
                     static_cast<size_t>(row) * a.row_stride * ElemTraits<DT>::kBytes;
    RowGeom g = make_geom<DT>(rp, a.V, S * kWarps);
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;
    pdl_wait();
    if (a.active && !a.active[row]) return;   // the whole cluster leaves together
    long p = 0;
    if (kPos) {
        p = a.pos[row];
        rp += p * a.pos_stride * ElemTraits<DT>::kBytes;
        g = make_geom<DT>(rp, a.V, S * kWarps);
    }
    float u = 0.f, ext = -1.f;
    if (!kGreedy && warp == 0) {   // fetched now, used after the stream
        if (a.ext_target) ext = fmaxf(__ldg(a.ext_target + row), 0.f);
        else u = __ldg(a.uniforms + (row + p * a.slot_stride));
    }
    const float thr = kThr ? a.thr[row] : neg_inf();
    Partial t = reduce_segment<DT, 2, kGreedy, kThr>(g, rank * kWarps + warp, a.c, lane, slot0, thr);
    if (lane == 0) { seg[warp].m = t.m; seg[warp].idx = t.idx; seg[warp].Z = t.Z; seg[warp].A = t.A; }
    cluster.sync();
    if (warp == 0) {
        Partial r; SegPick p;
        combine_segments<2>(cluster, seg, S, a.c, u, lane, r, p, ext);
        if (lane == 0) { res.row = r; res.pick = p; }
    }
    cluster_arrive();   // done with the peers' shared memory
    __syncthreads();    // res is visible block-wide
    const Partial R = res.row;
    const SegPick P = res.pick;
    const bool ok = (R.Z > 0.f) && (fabsf(R.m) <= kMaxLogit);
    // where this row's outputs live (the position is read again rather than kept across the stream)
    long slot = row;
    if (kPos && tid == 0) slot += a.pos[row] * a.slot_stride;
    if (rank == 0 && tid == 0) {
        float H = 0.f;
        if (ok) H = fmaxf(kLn2 * (log2f(R.Z) - R.A / R.Z), 0.f);
        else atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
        if (a.entropy) a.entropy[slot] = H;
        if (a.stop) a.stop[row] = __fsqrt_rn(H) > a.thresh ? 1 : 0;
        if (a.row_stats) { a.row_stats[2 * slot] = R.m; a.row_stats[2 * slot + 1] = R.Z; }
        if (kGreedy || !ok) a.token[slot] = ((R.idx >= 0 && R.idx < a.V) ? R.idx : 0) + a.token_offset;
    }
    if (!kGreedy && ok && P.seg / kWarps == rank) {
        SoftmaxWeights<DT> wf;
        wf.g = g; wf.c = a.c; wf.M = __fmul_rn(R.m, a.c); wf.thr = thr;
        int v_lo, v_hi;
        seg_range(g, P.seg, v_lo, v_hi);
        int virt = fine_scan<EPV>(wf, v_lo, v_hi, P.prefix, P.target, scan, tid, lane, warp);
        if (tid == 0) a.token[slot] = (virt >= 0 ? virt - g.pre : 0) + a.token_offset;
    }
    cluster_wait();     // no block leaves while a peer may still read its shared memory
}

// ------------------------------------------------------------------ row statistics (verify, phase 1)

struct StatsArgs {
    const void* logits;
    long row_stride;
    int V;
    float c;
    int draft_rows;          // 0: unit = row.  1: unit = (sequence, position) of a draft row
    int K;
    const int32_t* cu;
    long q_seq_stride, q_pos_stride;
    float2* out_stats;       // (m, Z) per row, indexed by target-row number
    int32_t* out_argmax;
    unsigned* status;
    float4* out_partial;     // kMode 2: (m, Z, A, index of the maximum + idx_offset as int bits)
    int idx_offset;
    const float* thr;        // kThr: truncation threshold per row (target rows: by target row; draft rows: by draft row)
};

template <int DT, int kMode, bool kThr = false>
__global__ void __launch_bounds__(kThreads) row_stats_kernel(StatsArgs a) {
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int unit = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ SegEntry seg[kWarps];
    extern __shared__ uint4 ring[];

    pdl_launch_dependents();
    pdl_wait();
    long in_row = unit;
    int out_row = unit;
    if (a.draft_rows) {
        int i = unit / a.K, j = unit - i * a.K;
        int row0 = a.cu ? a.cu[i] : i * (a.K + 1);
        int Ki = a.cu ? a.cu[i + 1] - row0 - 1 : a.K;
        if (j >= Ki) return;   // the whole cluster leaves together
        in_row = a.q_seq_stride < 0 ? static_cast<long>(row0 - i + j)
                                    : i * a.q_seq_stride + j * a.q_pos_stride;
        out_row = row0 + j;
    }
    const char* rp = static_cast<const char*>(a.logits) +
                     static_cast<size_t>(in_row) * a.row_stride * ElemTraits<DT>::kBytes;
    const RowGeom g = make_geom<DT>(rp, a.V, S * kWarps);
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;
    const float thr = kThr ? a.thr[in_row] : neg_inf();
    Partial t = reduce_segment<DT, kMode, kMode != 1, kThr>(g, rank * kWarps + warp, a.c, lane, slot0, thr);
    if (lane == 0) { seg[warp].m = t.m; seg[warp].idx = t.idx; seg[warp].Z = t.Z; seg[warp].A = t.A; }
    cluster.sync();
    if (rank == 0 && warp == 0) {
        Partial r; SegPick p;
        combine_segments<kMode>(cluster, seg, S, a.c, 0.f, lane, r, p);
        if (lane == 0) {
            bool ok = fabsf(r.m) <= kMaxLogit && (kMode == 0 || r.Z > 0.f);
            if (!ok && kMode != 2) atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);   // a shard may be all masked
            if (kMode == 1) a.out_stats[out_row] = make_float2(r.m, r.Z);
            if (kMode == 2) {
                int gi = ((r.idx >= 0 && r.idx < a.V) ? r.idx : 0) + a.idx_offset;
                a.out_partial[out_row] = make_float4(r.m, ok ? r.Z : 0.f, ok ? r.A : 0.f, __int_as_float(gi));
            }
            if (a.out_argmax) a.out_argmax[out_row] = (r.idx >= 0 && r.idx < a.V) ? r.idx : 0;
        }
    }
    cluster.sync();
}

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
};

// Weights max(0, p - q) of Algorithm 4 (or p alone for the bonus token) for one vector.
template <int DT>
struct ResidualWeights {
    RowGeom gt, gq;
    const void* qrow;
    float c, Mp, rZp, Mq, rZq;
    int bonus;
    float thr_p = -INFINITY, thr_q = -INFINITY;   // truncated distributions: logits below carry nothing
    __device__ __forceinline__ void operator()(int vi, float (&w)[ElemTraits<DT>::kEPV]) const {
        constexpr int EPV = ElemTraits<DT>::kEPV;
        float x[EPV];
        unpack_masked<DT>(__ldg(gt.base + vi), vi, gt, x);
#pragma unroll
        for (int j = 0; j < EPV; ++j)
            w[j] = x[j] >= thr_p ? ex2_approx(fmaxf(__fmaf_rn(x[j], c, -Mp), kArgFloor)) * rZp : 0.f;
        if (bonus) return;
        float d[EPV];
        if (gq.pre == gt.pre) {
            unpack_masked<DT>(__ldg(gq.base + vi), vi, gq, d);
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

struct FinishShared {
    int n_acc;
    SegPick pick;
};

template <int DT, bool kThr = false>
__global__ void __launch_bounds__(kThreads, 2) verify_finish_kernel(FinishArgs a) {
    using E = ElemTraits<DT>;
    constexpr int EPV = E::kEPV;
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
    if (warp == 0) {
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
                    // p(x)/q(x) = 2^(ap - aq) * Zq / Zp, from the difference of the two log2 arguments, so
                    // that a token however unlikely under both models keeps its ratio (no underflow)
                    const float ap = __fmaf_rn(tv, a.c, -__fmul_rn(ps.x, a.c));
                    const float aq = __fmaf_rn(dv, a.c, -__fmul_rn(qs.x, a.c));
                    bool p_zero = !(tv > neg_inf()), q_zero = !(dv > neg_inf());   // NaN counts as -inf
                    if (kThr) {   // tokens that the truncation dropped have probability zero
                        p_zero = p_zero || !(tv >= a.p_thr[row0 + j]);
                        q_zero = q_zero || !(dv >= a.q_thr[dr]);
                    }
                    // r < min(1, ratio) without the division: a ratio >= 1 accepts every r in [0,1);
                    // p(x) == 0 accepts none; q(x) == 0 < p(x) is a ratio of +inf
                    const float r = a.uniforms[row0 + j];
                    const float d = fminf(fmaxf(ap - aq, -126.f), 126.f);
                    const float num = __fmul_rn(exp2f(d), qs.y);
                    acc = !p_zero && (q_zero || num >= ps.y || __fmul_rn(r, ps.y) < num);
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
    const float u = a.uniforms[row0 + Ki];

    ResidualWeights<DT> wf;
    const char* trow = tl + static_cast<size_t>(row0 + n_acc) * a.t_row_stride * E::kBytes;
    wf.gt = make_geom<DT>(trow, a.V, S * kWarps);
    wf.c = a.c;
    {
        float2 ps = a.p_stats[row0 + n_acc];
        wf.Mp = __fmul_rn(ps.x, a.c);
        wf.rZp = 1.0f / ps.y;
        if (kThr) wf.thr_p = a.p_thr[row0 + n_acc];
    }
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

// ------------------------------------------------------------------ vocabulary-parallel draft step
//
// The vocabulary is sharded over G ranks (a tensor-parallel LM head).  Each rank reduces its shard of
// every row to (m, Z, A, argmax); the ranks exchange these 16 bytes per row; then every rank combines
// them in rank order -- same inputs, same arithmetic, so all ranks agree bit for bit on the entropy,
// the stop flag, and on which rank's shard holds the sampled token and how far into its mass.

struct VpCombineArgs {
    const float4* partials;   // [G][B]
    int G, B, rank;
    float c, thresh;
    int greedy;
    const float* uniforms;
    float* entropy;
    uint8_t* stop;
    int32_t* token;           // greedy: the global argmax; sampling: -1 (the owner fills it in)
    int32_t* owner;
    float* ext_target;
    uint8_t* active;
    unsigned* status;
};

__global__ void __launch_bounds__(kPolicyThreads) vp_combine_kernel(VpCombineArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * kPolicyThreads + threadIdx.x;
    if (b >= a.B) return;
    float m = neg_inf();
    for (int g = 0; g < a.G; ++g) m = fmaxf(m, a.partials[static_cast<size_t>(g) * a.B + b].x);
    const float M = __fmul_rn(m, a.c);
    float Z = 0.f, A = 0.f;
    int idx = kIntMax;
    for (int g = 0; g < a.G; ++g) {
        const float4 p = a.partials[static_cast<size_t>(g) * a.B + b];
        if (p.x == m) idx = min(idx, __float_as_int(p.w));
        if (p.y > 0.f) {
            float d = __fmul_rn(p.x, a.c) - M;
            float s = ex2_approx(fmaxf(d, kArgFloor));
            A += s * __fmaf_rn(d, p.y, p.z);
            Z += s * p.y;
        }
    }
    const bool ok = Z > 0.f && fabsf(m) <= kMaxLogit;
    float H = 0.f;
    if (ok) H = fmaxf(kLn2 * (log2f(Z) - A / Z), 0.f);
    else atomicOr(a.status, SVIP_STATUS_NONFINITE_ROW);
    a.entropy[b] = H;
    a.stop[b] = __fsqrt_rn(H) > a.thresh ? 1 : 0;
    int owner = -1;
    float local_target = 0.f;
    if (!a.greedy && ok) {
        const float target = a.uniforms[b] * Z;
        float run = 0.f, before = 0.f;
        int last = -1;
        for (int g = 0; g < a.G && owner < 0; ++g) {
            const float4 p = a.partials[static_cast<size_t>(g) * a.B + b];
            float mass = 0.f;
            if (p.y > 0.f) mass = p.y * ex2_approx(fmaxf(__fmul_rn(p.x, a.c) - M, kArgFloor));
            if (mass > 0.f) {
                last = g; before = run;
                if (run + mass > target) owner = g;
            }
            run += mass;
        }
        if (owner < 0) owner = last;   // rounding: the last shard with mass, searched to its end
        // the owner looks for (target - before) in units of its own Z, i.e. relative to its own maximum
        const float4 po = a.partials[static_cast<size_t>(owner) * a.B + b];
        const float up = ex2_approx(fminf(M - __fmul_rn(po.x, a.c), 126.f));
        local_target = fminf(fmaxf(target - before, 0.f) * up, po.y);
    }
    a.token[b] = a.greedy || !ok ? ((idx != kIntMax) ? idx : 0) : -1;
    a.owner[b] = owner;
    a.ext_target[b] = local_target;
    a.active[b] = owner == a.rank ? 1 : 0;
}

// ------------------------------------------------------------------ draft-length policies
//
// Per-sequence drafting state on the device, so that the loop of Algorithm 1 needs no host round
// trip per draft token.  ENTROPY is the paper's rule (Eq. 7 flag from the draft step); CONSTANT and
// HEURISTIC are the two baselines of Section 3.

// Control of a drafting loop recorded as a WHILE node of a CUDA graph.  The kernel that closes an
// iteration counts it and tells the graph whether the body runs again: only while sequences are
// still drafting, and never more than `max_iters` times whatever the data say.
struct LoopCtl {
    cudaGraphConditionalHandle handle;
    int* iter;        // iterations done since the loop was entered (NULL: not inside a loop)
    int max_iters;
};

__device__ __forceinline__ void loop_decide(const LoopCtl& loop, int n_active) {
    if (!loop.iter) return;
    const int it = *loop.iter + 1;
    *loop.iter = it;
    cudaGraphSetConditional(loop.handle, (n_active > 0 && it < loop.max_iters) ? 1u : 0u);
}

struct AdvanceArgs {
    int policy;
    const uint8_t* stop;
    const int32_t* gamma;
    int32_t* draft_len;
    uint8_t* active;
    int B, K_cap;
    int32_t* n_active;
    LoopCtl loop;
};

__global__ void __launch_bounds__(kPolicyThreads) policy_advance_kernel(AdvanceArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    // one block: counts the sequences still drafting while it updates them
    __shared__ int count;
    if (threadIdx.x == 0) count = 0;
    __syncthreads();
    int mine = 0;
    for (int i = threadIdx.x; i < a.B; i += kPolicyThreads) {
        if (!a.active[i]) continue;
        int len = a.draft_len[i] + 1;
        a.draft_len[i] = len;
        bool done;
        if (a.policy == SVIP_POLICY_ENTROPY) done = a.stop[i] != 0 || len >= a.K_cap;
        else done = len >= min(a.gamma[i], a.K_cap);
        if (done) a.active[i] = 0; else ++mine;
    }
    if (mine) atomicAdd(&count, mine);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (a.n_active) *a.n_active = count;
        loop_decide(a.loop, count);
    }
}

// Decision of a drafting loop whose body holds no svip_policy_advance on the loop's counter.
__global__ void loop_decide_kernel(LoopCtl loop, const int32_t* n_active) {
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) loop_decide(loop, *n_active);
}

struct UpdateArgs {
    int policy;
    const int32_t* n_accepted;
    int32_t* draft_len;
    int32_t* gamma;
    uint8_t* active;
    int B, K_cap;
};

__global__ void __launch_bounds__(kPolicyThreads) policy_update_kernel(UpdateArgs a) {
    pdl_launch_dependents();
    pdl_wait();
    int i = blockIdx.x * kPolicyThreads + threadIdx.x;
    if (i >= a.B) return;
    if (a.policy == SVIP_POLICY_HEURISTIC) {
        int g = a.gamma[i];
        g = a.n_accepted[i] == a.draft_len[i] ? min(g + 2, a.K_cap) : max(g - 1, 1);
        a.gamma[i] = g;
    }
    a.draft_len[i] = 0;
    a.active[i] = 1;
}

// ------------------------------------------------------------------ ragged packing

constexpr int kPackThreads = 1024;

__global__ void __launch_bounds__(kPackThreads) pack_ragged_kernel(const int32_t* draft_len, int B, int K_max,
                                                                   int32_t* cu, int32_t* row_seq,
                                                                   int32_t* row_pos, unsigned* status) {
    __shared__ int wsum[32];
    __shared__ int carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    pdl_wait();
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < B; base += kPackThreads) {
        int i = base + tid;
        int k = 0;
        if (i < B) {
            k = draft_len[i];
            if (k < 1 || k > K_max) {
                atomicOr(status, SVIP_STATUS_BAD_DRAFT_LEN);
                k = k < 1 ? 1 : K_max;
            }
            k += 1;
        }
        int inc = k;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += n;
        }
        if (lane == 31) wsum[warp] = inc;
        __syncthreads();
        int before = 0, tot = 0;
        for (int w = 0; w < 32; ++w) {
            int s = wsum[w];
            if (w < warp) before += s;
            tot += s;
        }
        int c0 = carry;
        if (i < B) cu[i] = c0 + before + inc - k;
        __syncthreads();
        if (tid == 0) carry = c0 + tot;
        __syncthreads();
    }
    const int total = carry;
    if (tid == 0) cu[B] = total;
    __syncthreads();
    if (row_seq || row_pos) {
        for (int r = tid; r < total; r += kPackThreads) {
            int lo = 0, hi = B;           // largest i with cu[i] <= r
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if (cu[mid] <= r) lo = mid; else hi = mid;
            }
            if (row_seq) row_seq[r] = lo;
            if (row_pos) row_pos[r] = r - cu[lo];
        }
    }
}

}  // namespace svip

#include "svip_select.cuh"

// ==================================================================== host side / C ABI

using namespace svip;

struct svip_ctx {
    int device;
    int max_rows;
    int num_sms;
    int cluster_override;
    long launches;
    int last_cuda;
    int capturing;
    float2* p_stats;
    float2* q_stats;
    int32_t* p_argmax;
    unsigned* status;
    uint8_t* need;             // device [max_rows]: rows that svip_draft_step_truncated leaves to the streaming kernel
    int* loop_iter;            // device: iteration counter of the drafting loop being replayed
    cudaStream_t loop_stream;  // records the body of a drafting loop
    int loop_open;             // a loop body is being recorded
    int loop_decided;          // the body already holds the kernel that decides the loop
    int loop_failed;           // a loop of the graph being recorded is not closed properly
    LoopCtl loop;
    const int32_t* loop_n_active;
    int profiling;
    int prof_used;
    cudaEvent_t* prof_start;
    cudaEvent_t* prof_stop;
};

constexpr int kProfilePairs = 4096;

struct svip_graph {
    cudaGraphExec_t exec;
    cudaGraph_t graph;
};

namespace {

// SVIP_NO_PDL=1 in the environment launches every kernel fully serialized (for A/B timing).
const bool g_use_pdl = [] {
    const char* v = std::getenv("SVIP_NO_PDL");
    return !(v && v[0] == '1');
}();

// Set while the calling thread records the body of a drafting loop: kernels inside a conditional
// node are launched without the programmatic-serialization attribute.
thread_local bool t_plain_launches = false;

int cuda_fail(svip_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda = static_cast<int>(e);
    return SVIP_ERR_CUDA;
}

// Every kernel goes through here: optional cluster dimension, dynamic shared memory, and the
// programmatic-serialization attribute that lets the kernel be scheduled while its predecessor in
// the stream drains (the kernels wait for the predecessor themselves, see pdl_wait()).
template <class... KArgs, class... Args>
cudaError_t launch_ex(void (*kernel)(KArgs...), unsigned grid, unsigned block, int S, size_t dyn_smem,
                      cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = dyn_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (S > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = S;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (g_use_pdl && !t_plain_launches) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <class Args>
cudaError_t launch_clustered(void (*kernel)(Args), long units, int S, const Args& args, cudaStream_t st,
                             size_t dyn_smem) {
    return launch_ex(kernel, static_cast<unsigned>(units * S), kThreads, S, dyn_smem, st, args);
}

// Blocks per row.  Small launches are latency-bound: spread a row over as many blocks (1..8, any
// size) as still lets the whole grid sit on the GPU at once (two blocks per SM) while every thread
// keeps a vector; a second wave of clusters would double the time of such a launch.
int pick_cluster(const svip_ctx* ctx, long rows, int V, int dtype) {
    if (ctx->cluster_override > 0) return ctx->cluster_override;
    long nvec = (static_cast<long>(V) * (dtype == SVIP_BF16 ? 2 : 4) + 15) / 16;
    // measured: grids up to about 7/4 blocks per SM run as one wave next to the blocks of the
    // following launch that programmatic launch makes resident early; fuller grids run as two
    long by_grid = rows > 0 ? (7L * ctx->num_sms / 4) / rows : kMaxCluster;
    long by_work = nvec / kThreads;
    long S = by_grid < by_work ? by_grid : by_work;
    if (S > kMaxCluster) S = kMaxCluster;
    if (S < 1) S = 1;
    // many long rows (more than a wave of blocks anyway): rows above 512 KB are cut so that the
    // two blocks of an SM finish close together (measured on 256 x 1 MB: 64 -> 55 us)
    const long row_bytes = nvec * 16;
    if (S == 1 && rows > ctx->num_sms && row_bytes > (512L << 10)) {
        S = (row_bytes + (512L << 10) - 1) / (512L << 10);
        if (S > 4) S = 4;
    }
    return static_cast<int>(S);
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

float scale_for(float T) { return static_cast<float>(1.4426950408889634 / (T > 0.f ? static_cast<double>(T) : 1.0)); }

}  // namespace

extern "C" {

const char* svip_strerror(int status) {
    switch (status) {
        case SVIP_OK: return "ok";
        case SVIP_ERR_INVALID_ARG: return "invalid argument";
        case SVIP_ERR_UNSUPPORTED: return "unsupported dtype or device";
        case SVIP_ERR_WORKSPACE: return "more rows than the context's workspace holds";
        case SVIP_ERR_CUDA: return "CUDA runtime error";
        case SVIP_ERR_STATE: return "call not valid in the context's current state";
        default: return "unknown status";
    }
}

int svip_version(void) { return 200; }

int svip_last_cuda_error(const svip_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

int svip_create(svip_ctx** out, int device, int max_rows) {
    if (!out || max_rows < 1 || device < 0) return SVIP_ERR_INVALID_ARG;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
    int rc = SVIP_OK;
    svip_ctx* c = new (std::nothrow) svip_ctx();
    if (!c) { cudaSetDevice(prev); return SVIP_ERR_CUDA; }
    c->device = device;
    c->max_rows = max_rows;
    int major = 0, sms = 0;
    cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) rc = SVIP_ERR_CUDA;
    else if (major != 10) rc = SVIP_ERR_UNSUPPORTED;
    c->num_sms = sms;
    if (rc == SVIP_OK) {
        // the cp.async rings need more dynamic shared memory than the default limit
        const void* ringed[] = {
            (const void*)draft_step_kernel<kBF16, true, 2>, (const void*)draft_step_kernel<kBF16, false, 2>,
            (const void*)draft_step_kernel<kF32, true, 2>,  (const void*)draft_step_kernel<kF32, false, 2>,
            (const void*)draft_step_kernel<kBF16, true, 3>, (const void*)draft_step_kernel<kBF16, false, 3>,
            (const void*)draft_step_kernel<kF32, true, 3>,  (const void*)draft_step_kernel<kF32, false, 3>,
            (const void*)draft_step_kernel<kBF16, true, 2, true>, (const void*)draft_step_kernel<kBF16, false, 2, true>,
            (const void*)draft_step_kernel<kF32, true, 2, true>,  (const void*)draft_step_kernel<kF32, false, 2, true>,
            (const void*)row_stats_kernel<kBF16, 0>,     (const void*)row_stats_kernel<kBF16, 1>,
            (const void*)row_stats_kernel<kF32, 0>,      (const void*)row_stats_kernel<kF32, 1>,
            (const void*)verify_finish_kernel<kBF16>,    (const void*)verify_finish_kernel<kF32>,
            (const void*)row_stats_kernel<kBF16, 2>,     (const void*)row_stats_kernel<kF32, 2>,
            (const void*)row_threshold_kernel<kBF16>,    (const void*)row_threshold_kernel<kF32>,
            (const void*)row_threshold_kernel<kBF16, true>, (const void*)row_threshold_kernel<kF32, true>,
            (const void*)draft_step_kernel<kBF16, false, 2, false, true>, (const void*)draft_step_kernel<kF32, false, 2, false, true>,
            (const void*)row_stats_kernel<kBF16, 1, true>, (const void*)row_stats_kernel<kF32, 1, true>,
            (const void*)verify_finish_kernel<kBF16, true>, (const void*)verify_finish_kernel<kF32, true>};
        for (const void* k : ringed)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes) != cudaSuccess)
                rc = SVIP_ERR_CUDA;
    }
    if (rc == SVIP_OK) {
        size_t n = static_cast<size_t>(max_rows);
        if (cudaMalloc(&c->p_stats, n * sizeof(float2)) != cudaSuccess ||
            cudaMalloc(&c->q_stats, n * sizeof(float2)) != cudaSuccess ||
            cudaMalloc(&c->p_argmax, n * sizeof(int32_t)) != cudaSuccess ||
            cudaMalloc(&c->status, sizeof(unsigned)) != cudaSuccess ||
            cudaMemset(c->status, 0, sizeof(unsigned)) != cudaSuccess ||
            cudaMalloc(&c->need, n) != cudaSuccess ||
            cudaMalloc(&c->loop_iter, sizeof(int)) != cudaSuccess ||
            cudaMemset(c->loop_iter, 0, sizeof(int)) != cudaSuccess) {
            rc = SVIP_ERR_CUDA;
        }
    }
    if (rc != SVIP_OK) {
        cudaGetLastError();
        cudaFree(c->p_stats); cudaFree(c->q_stats); cudaFree(c->p_argmax); cudaFree(c->status);
        cudaFree(c->loop_iter); cudaFree(c->need);
        delete c;
    } else {
        *out = c;
    }
    cudaSetDevice(prev);
    return rc;
}

int svip_destroy(svip_ctx* ctx) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    cudaFree(ctx->p_stats); cudaFree(ctx->q_stats); cudaFree(ctx->p_argmax); cudaFree(ctx->status);
    cudaFree(ctx->loop_iter); cudaFree(ctx->need);
    if (ctx->loop_stream) cudaStreamDestroy(ctx->loop_stream);
    if (ctx->prof_start) {
        for (int k = 0; k < kProfilePairs; ++k) {
            cudaEventDestroy(ctx->prof_start[k]);
            cudaEventDestroy(ctx->prof_stop[k]);
        }
        delete[] ctx->prof_start;
        delete[] ctx->prof_stop;
    }
    cudaSetDevice(prev);
    delete ctx;
    return SVIP_OK;
}

int svip_set_cluster_size(svip_ctx* ctx, int cluster_size) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (cluster_size < 0 || cluster_size > kMaxCluster) return SVIP_ERR_INVALID_ARG;
    ctx->cluster_override = cluster_size;
    return SVIP_OK;
}

long svip_launch_count(const svip_ctx* ctx) { return ctx ? ctx->launches : 0; }

int svip_read_status(svip_ctx* ctx, unsigned* flags, void* stream) {
    if (!ctx || !flags) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, ctx->status, sizeof v, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof v, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    *flags = v;
    return SVIP_OK;
}

static int draft_impl(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                      long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                      const float* uniforms, const uint8_t* active, const float* thr, int32_t* token,
                      float* entropy, uint8_t* stop, float* row_stats, void* stream);

int svip_draft_step(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                    float T, float thresh, const float* uniforms, int32_t* token, float* entropy,
                    uint8_t* stop, float* row_stats, void* stream) {
    return svip_draft_step_masked(ctx, logits, dtype, B, V, row_stride, T, thresh, uniforms, nullptr, token,
                                  entropy, stop, row_stats, stream);
}

int svip_draft_step_masked(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                           float T, float thresh, const float* uniforms, const uint8_t* active,
                           int32_t* token, float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    return svip_draft_step_at(ctx, logits, dtype, B, V, row_stride, 0, nullptr, 0, T, thresh, uniforms, active,
                              token, entropy, stop, row_stats, stream);
}

int svip_draft_step_at(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                       long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                       const float* uniforms, const uint8_t* active, int32_t* token, float* entropy,
                       uint8_t* stop, float* row_stats, void* stream) {
    return draft_impl(ctx, logits, dtype, B, V, row_stride, pos_stride, pos, slot_stride, T, thresh, uniforms, active,
                      nullptr, token, entropy, stop, row_stats, stream);
}

int svip_draft_step_filtered(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                             float T, float thresh, const float* uniforms, const uint8_t* active, const float* thr,
                             int32_t* token, float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    if (!thr || !(T > 0.f)) return SVIP_ERR_INVALID_ARG;
    return draft_impl(ctx, logits, dtype, B, V, row_stride, 0, nullptr, 0, T, thresh, uniforms, active, thr, token,
                      entropy, stop, row_stats, stream);
}

static int draft_impl(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                      long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                      const float* uniforms, const uint8_t* active, const float* thr, int32_t* token,
                      float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    if (!ctx || !logits || !token || !entropy || !stop) return SVIP_ERR_INVALID_ARG;
    if (pos_stride < 0 || slot_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T) || std::isnan(thresh)) return SVIP_ERR_INVALID_ARG;
    if (T > 0.f && !uniforms) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    DraftArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T); a.thresh = thresh;
    a.greedy = T > 0.f ? 0 : 1; a.uniforms = uniforms; a.token = token; a.entropy = entropy;
    a.stop = stop; a.row_stats = row_stats; a.status = ctx->status; a.active = active;
    a.ext_target = nullptr; a.token_offset = 0;
    a.pos = pos; a.pos_stride = pos_stride; a.slot_stride = slot_stride; a.thr = thr;
    int S = pick_cluster(ctx, B, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool waves = static_cast<long>(B) * S > 2L * ctx->num_sms;
    void (*k)(DraftArgs);
    if (dtype == SVIP_BF16)
        k = a.greedy ? (waves ? draft_step_kernel<kBF16, true, 3> : draft_step_kernel<kBF16, true, 2>)
                     : (waves ? draft_step_kernel<kBF16, false, 3> : draft_step_kernel<kBF16, false, 2>);
    else
        k = a.greedy ? (waves ? draft_step_kernel<kF32, true, 3> : draft_step_kernel<kF32, true, 2>)
                     : (waves ? draft_step_kernel<kF32, false, 3> : draft_step_kernel<kF32, false, 2>);
    if (pos) {
        if (dtype == SVIP_BF16) k = a.greedy ? draft_step_kernel<kBF16, true, 2, true> : draft_step_kernel<kBF16, false, 2, true>;
        else k = a.greedy ? draft_step_kernel<kF32, true, 2, true> : draft_step_kernel<kF32, false, 2, true>;
    }
    if (thr) k = dtype == SVIP_BF16 ? draft_step_kernel<kBF16, false, 2, false, true> : draft_step_kernel<kF32, false, 2, false, true>;
    cudaError_t e = launch_clustered(k, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_row_threshold(svip_ctx* ctx, const void* logits, svip_dtype dtype, int n_rows, int V, long row_stride,
                       float T, int top_k, float top_p, float* thr, float* stats, void* stream) {
    if (!ctx || !logits || !thr) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (n_rows < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0 || top_k < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(top_p > 0.f)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (n_rows == 0) return SVIP_OK;
    ThresholdArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T);
    a.top_k = (top_k >= 1 && top_k < V) ? top_k : 0; a.top_p = top_p; a.thr = thr;
    a.stats = reinterpret_cast<float2*>(stats);
    if (stats && !aligned_to(stats, 8)) return SVIP_ERR_INVALID_ARG;
    a.uniforms = nullptr; a.active = nullptr; a.thresh = 0.f; a.token = nullptr; a.entropy = nullptr;
    a.stop = nullptr; a.need = nullptr;
    const int S = pick_cluster(ctx, n_rows, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(row_threshold_kernel<kBF16>, n_rows, S, a, st, kRingBytes)
                                       : launch_clustered(row_threshold_kernel<kF32>, n_rows, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_draft_step_truncated(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                              float T, float thresh, int top_k, float top_p, const float* uniforms,
                              const uint8_t* active, float* thr, int32_t* token, float* entropy, uint8_t* stop,
                              float* row_stats, void* stream) {
    if (!ctx || !logits || !thr || !token || !entropy || !stop || !uniforms) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0 || top_k < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(top_p > 0.f) || std::isnan(thresh)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (row_stats && !aligned_to(row_stats, 8)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    if (B > ctx->max_rows) return SVIP_ERR_WORKSPACE;
    ThresholdArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T);
    a.top_k = (top_k >= 1 && top_k < V) ? top_k : 0; a.top_p = top_p; a.thr = thr;
    a.stats = reinterpret_cast<float2*>(row_stats);
    a.uniforms = uniforms; a.active = active; a.thresh = thresh; a.token = token; a.entropy = entropy;
    a.stop = stop; a.need = ctx->need;
    const int S = pick_cluster(ctx, B, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16
        ? launch_clustered(row_threshold_kernel<kBF16, true>, B, S, a, st, kRingBytes)
        : launch_clustered(row_threshold_kernel<kF32, true>, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    // the rows the candidates could not finish: the streaming draft step at the thresholds just found
    return svip_draft_step_filtered(ctx, logits, dtype, B, V, row_stride, T, thresh, uniforms, ctx->need, thr, token,
                                    entropy, stop, row_stats, stream);
}

int svip_pack_ragged(svip_ctx* ctx, const int32_t* draft_len, int B, int K_max, int32_t* cu_rows,
                     int32_t* row_seq, int32_t* row_pos, void* stream) {
    if (!ctx || !draft_len || !cu_rows) return SVIP_ERR_INVALID_ARG;
    if (B < 1 || B > 65536 || K_max < 1) return SVIP_ERR_INVALID_ARG;
    if (static_cast<long>(B) * (static_cast<long>(K_max) + 1) >= 0x7fffffffL) return SVIP_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_ex(pack_ragged_kernel, 1, kPackThreads, 0, 0, st, draft_len, B, K_max, cu_rows, row_seq,
                              row_pos, ctx->status);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

// The verification round; q_thr / p_thr are both NULL (plain distributions) or both given
// (distributions truncated at those per-row thresholds).
static int verify_impl(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                       const float* q_stats, long q_seq_stride, long q_pos_stride, const void* target_logits,
                       long t_row_stride, svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                       int n_target_rows, int V, float T, const float* uniforms, int32_t* n_accepted,
                       int32_t* next_token, void* stream, const float* q_thr, const float* p_thr,
                       const float* p_stats_user) {
    if (!ctx || !draft_tokens || !target_logits || !n_accepted || !next_token) return SVIP_ERR_INVALID_ARG;
    const bool truncated = q_thr != nullptr;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || K < 1 || V < 1 || V > 0x7fffffe0 || t_row_stride < 0 || q_row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    const bool sampling = T > 0.f;
    if (sampling && (!q_logits || !uniforms)) return SVIP_ERR_INVALID_ARG;
    if (q_seq_stride < 0 && q_seq_stride != SVIP_Q_PACKED) return SVIP_ERR_INVALID_ARG;
    if (q_seq_stride >= 0 && q_pos_stride < 0) return SVIP_ERR_INVALID_ARG;
    const size_t esz = dtype == SVIP_BF16 ? 2 : 4;
    if (!aligned_to(target_logits, esz) || (q_logits && !aligned_to(q_logits, esz))) return SVIP_ERR_INVALID_ARG;
    if (static_cast<long>(B) * (static_cast<long>(K) + 1) >= 0x7fffffffL) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return n_target_rows == 0 ? SVIP_OK : SVIP_ERR_INVALID_ARG;
    if (n_target_rows < 2 * B || n_target_rows > B * (K + 1)) return SVIP_ERR_INVALID_ARG;
    if (!cu_rows && n_target_rows != B * (K + 1)) return SVIP_ERR_INVALID_ARG;
    if (n_target_rows > ctx->max_rows) return SVIP_ERR_WORKSPACE;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float c = scale_for(T);
    cudaError_t e;

    StatsArgs s;
    s.logits = target_logits; s.row_stride = t_row_stride; s.V = V; s.c = c; s.draft_rows = 0; s.K = K;
    s.cu = cu_rows; s.q_seq_stride = q_seq_stride; s.q_pos_stride = q_pos_stride;
    s.out_stats = ctx->p_stats; s.out_argmax = sampling ? nullptr : ctx->p_argmax; s.status = ctx->status;
    s.out_partial = nullptr; s.idx_offset = 0; s.thr = p_thr;
    int S = pick_cluster(ctx, n_target_rows, V, dtype);
    const bool timed = ctx->profiling && !ctx->capturing && ctx->prof_used < kProfilePairs;
    if (timed) cudaEventRecord(ctx->prof_start[ctx->prof_used], st);
    if (p_stats_user)
        e = cudaSuccess;   // the caller already holds (m, Z) of every target row
    else if (truncated)
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1, true>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1, true>, n_target_rows, S, s, st, kRingBytes);
    else if (sampling)
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1>, n_target_rows, S, s, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 0>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 0>, n_target_rows, S, s, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (!p_stats_user) ctx->launches += 1;
    if (timed) cudaEventRecord(ctx->prof_stop[ctx->prof_used++], st);

    if (!sampling) {
        GreedyArgs g;
        g.draft_tokens = draft_tokens; g.p_argmax = ctx->p_argmax; g.cu = cu_rows;
        g.q_seq_stride = q_seq_stride; g.q_pos_stride = q_pos_stride; g.B = B; g.K = K;
        g.n_accepted = n_accepted; g.next_token = next_token;
        e = launch_ex(verify_greedy_kernel, static_cast<unsigned>((B + kWarps - 1) / kWarps), kThreads, 0, 0, st, g);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
        return SVIP_OK;
    }

    if (!q_stats) {
        StatsArgs d = s;
        d.logits = q_logits; d.row_stride = q_row_stride; d.draft_rows = 1;
        d.out_stats = ctx->q_stats; d.out_argmax = nullptr; d.thr = q_thr;
        long units = static_cast<long>(B) * K;
        int Sd = pick_cluster(ctx, n_target_rows - B, V, dtype);
        if (truncated)
            e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1, true>, units, Sd, d, st, kRingBytes)
                                   : launch_clustered(row_stats_kernel<kF32, 1, true>, units, Sd, d, st, kRingBytes);
        else
            e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, units, Sd, d, st, kRingBytes)
                                   : launch_clustered(row_stats_kernel<kF32, 1>, units, Sd, d, st, kRingBytes);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }

    FinishArgs f;
    f.draft_tokens = draft_tokens; f.q_logits = q_logits; f.q_row_stride = q_row_stride;
    f.q_stats_user = reinterpret_cast<const float2*>(q_stats); f.q_stats_ws = ctx->q_stats;
    f.q_seq_stride = q_seq_stride; f.q_pos_stride = q_pos_stride; f.t_logits = target_logits;
    f.t_row_stride = t_row_stride;
    f.p_stats = p_stats_user ? reinterpret_cast<const float2*>(p_stats_user) : ctx->p_stats;
    f.cu = cu_rows; f.K = K; f.V = V; f.c = c;
    f.uniforms = uniforms; f.n_accepted = n_accepted; f.next_token = next_token; f.status = ctx->status;
    f.p_thr = p_thr; f.q_thr = q_thr;
    // up to two rows per sequence are streamed: long rows are cut finer than the one-wave policy
    // asks for (this kernel runs for many microseconds, so several waves are fine)
    int Sf = pick_cluster(ctx, B, V, dtype);
    if (ctx->cluster_override == 0) {
        const long row_bytes = static_cast<long>(V) * static_cast<long>(esz);
        while (Sf < kMaxCluster && 2 * row_bytes / Sf > (512L << 10)) Sf *= 2;
        if (Sf > kMaxCluster) Sf = kMaxCluster;
    }
    if (truncated)
        e = dtype == SVIP_BF16 ? launch_clustered(verify_finish_kernel<kBF16, true>, B, Sf, f, st, kRingBytes)
                               : launch_clustered(verify_finish_kernel<kF32, true>, B, Sf, f, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(verify_finish_kernel<kBF16>, B, Sf, f, st, kRingBytes)
                               : launch_clustered(verify_finish_kernel<kF32>, B, Sf, f, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_verify(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                const float* q_stats, long q_seq_stride, long q_pos_stride, const void* target_logits,
                long t_row_stride, svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                int n_target_rows, int V, float T, const float* uniforms, int32_t* n_accepted,
                int32_t* next_token, void* stream) {
    return verify_impl(ctx, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream, nullptr, nullptr, nullptr);
}

int svip_verify_filtered(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                         const float* q_stats, const float* q_thr, long q_seq_stride, long q_pos_stride,
                         const void* target_logits, long t_row_stride, const float* p_thr, const float* p_stats,
                         svip_dtype dtype, const int32_t* cu_rows, int B, int K, int n_target_rows, int V, float T,
                         const float* uniforms, int32_t* n_accepted, int32_t* next_token, void* stream) {
    if (!q_thr || !p_thr || !(T > 0.f)) return SVIP_ERR_INVALID_ARG;
    if (p_stats && !aligned_to(p_stats, 8)) return SVIP_ERR_INVALID_ARG;
    return verify_impl(ctx, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream, q_thr, p_thr, p_stats);
}

int svip_profile_enable(svip_ctx* ctx, int on) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    if (on && !ctx->prof_start) {
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(ctx->device);
        ctx->prof_start = new (std::nothrow) cudaEvent_t[kProfilePairs]();
        ctx->prof_stop = new (std::nothrow) cudaEvent_t[kProfilePairs]();
        cudaError_t e = (ctx->prof_start && ctx->prof_stop) ? cudaSuccess : cudaErrorMemoryAllocation;
        for (int k = 0; k < kProfilePairs && e == cudaSuccess; ++k) {
            e = cudaEventCreate(&ctx->prof_start[k]);
            if (e == cudaSuccess) e = cudaEventCreate(&ctx->prof_stop[k]);
        }
        cudaSetDevice(prev);
        if (e != cudaSuccess) {
            delete[] ctx->prof_start; delete[] ctx->prof_stop;   // events created so far leak with the context
            ctx->prof_start = ctx->prof_stop = nullptr;
            return cuda_fail(ctx, e);
        }
    }
    ctx->profiling = on ? 1 : 0;
    ctx->prof_used = 0;
    return SVIP_OK;
}

int svip_profile_read(svip_ctx* ctx, double* total_ms, long* launches) {
    if (!ctx || !total_ms || !launches) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    double sum = 0.0;
    for (int k = 0; k < ctx->prof_used; ++k) {
        cudaError_t e = cudaEventSynchronize(ctx->prof_stop[k]);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->prof_start[k], ctx->prof_stop[k]);
        if (e != cudaSuccess) { ctx->prof_used = 0; return cuda_fail(ctx, e); }
        sum += ms;
    }
    *total_ms = sum;
    *launches = ctx->prof_used;
    ctx->prof_used = 0;
    return SVIP_OK;
}

int svip_policy_advance(svip_ctx* ctx, int policy, const uint8_t* stop, const int32_t* gamma,
                        int32_t* draft_len, uint8_t* active, int B, int K_cap, int32_t* n_active,
                        void* stream) {
    if (!ctx || !draft_len || !active || B < 0 || K_cap < 1) return SVIP_ERR_INVALID_ARG;
    if (policy != SVIP_POLICY_ENTROPY && policy != SVIP_POLICY_CONSTANT && policy != SVIP_POLICY_HEURISTIC)
        return SVIP_ERR_INVALID_ARG;
    if (policy == SVIP_POLICY_ENTROPY ? !stop : !gamma) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    AdvanceArgs a;
    a.policy = policy; a.stop = stop; a.gamma = gamma; a.draft_len = draft_len; a.active = active;
    a.B = B; a.K_cap = K_cap; a.n_active = n_active;
    a.loop.iter = nullptr; a.loop.max_iters = 0; a.loop.handle = 0;
    const bool decides = ctx->loop_open && n_active && n_active == ctx->loop_n_active &&
                         static_cast<cudaStream_t>(stream) == ctx->loop_stream;
    if (decides) a.loop = ctx->loop;
    cudaError_t e = launch_ex(policy_advance_kernel, 1, kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (decides) ctx->loop_decided = 1;
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_policy_update(svip_ctx* ctx, int policy, const int32_t* n_accepted, int32_t* draft_len,
                       int32_t* gamma, uint8_t* active, int B, int K_cap, void* stream) {
    if (!ctx || !draft_len || !active || B < 0 || K_cap < 1) return SVIP_ERR_INVALID_ARG;
    if (policy != SVIP_POLICY_ENTROPY && policy != SVIP_POLICY_CONSTANT && policy != SVIP_POLICY_HEURISTIC)
        return SVIP_ERR_INVALID_ARG;
    if (policy == SVIP_POLICY_HEURISTIC && (!gamma || !n_accepted)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    UpdateArgs a;
    a.policy = policy; a.n_accepted = n_accepted; a.draft_len = draft_len; a.gamma = gamma; a.active = active;
    a.B = B; a.K_cap = K_cap;
    cudaError_t e = launch_ex(policy_update_kernel, static_cast<unsigned>((B + kPolicyThreads - 1) / kPolicyThreads),
                              kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_partial(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard, long row_stride,
                    float T, int vocab_offset, float* partial, void* stream) {
    if (!ctx || !logits || !partial) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V_shard < 1 || V_shard > 0x7fffffe0 || row_stride < 0 || vocab_offset < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4) || !aligned_to(partial, 16)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    StatsArgs s;
    s.logits = logits; s.row_stride = row_stride; s.V = V_shard; s.c = scale_for(T); s.draft_rows = 0; s.K = 1;
    s.cu = nullptr; s.q_seq_stride = 0; s.q_pos_stride = 0; s.out_stats = nullptr; s.out_argmax = nullptr;
    s.status = ctx->status; s.out_partial = reinterpret_cast<float4*>(partial); s.idx_offset = vocab_offset;
    const int S = pick_cluster(ctx, B, V_shard, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 2>, B, S, s, st, kRingBytes)
                                       : launch_clustered(row_stats_kernel<kF32, 2>, B, S, s, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_combine(svip_ctx* ctx, const float* partials, int G, int rank, int B, float T, float thresh,
                    const float* uniforms, float* entropy, uint8_t* stop, int32_t* token, int32_t* owner,
                    float* local_target, uint8_t* active, void* stream) {
    if (!ctx || !partials || !entropy || !stop || !token || !owner || !local_target || !active)
        return SVIP_ERR_INVALID_ARG;
    if (G < 1 || rank < 0 || rank >= G || B < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T) || std::isnan(thresh) || (T > 0.f && !uniforms)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(partials, 16)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    VpCombineArgs a;
    a.partials = reinterpret_cast<const float4*>(partials); a.G = G; a.B = B; a.rank = rank; a.c = scale_for(T);
    a.thresh = thresh; a.greedy = T > 0.f ? 0 : 1; a.uniforms = uniforms; a.entropy = entropy; a.stop = stop;
    a.token = token; a.owner = owner; a.ext_target = local_target; a.active = active; a.status = ctx->status;
    cudaError_t e = launch_ex(vp_combine_kernel, static_cast<unsigned>((B + kPolicyThreads - 1) / kPolicyThreads),
                              kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_locate(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard, long row_stride,
                   float T, const float* local_target, const uint8_t* active, int vocab_offset,
                   int32_t* token, void* stream) {
    if (!ctx || !logits || !local_target || !active || !token) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V_shard < 1 || V_shard > 0x7fffffe0 || row_stride < 0 || vocab_offset < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    DraftArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V_shard; a.c = scale_for(T); a.thresh = 0.f; a.greedy = 0;
    a.uniforms = nullptr; a.token = token; a.entropy = nullptr; a.stop = nullptr; a.row_stats = nullptr;
    a.status = ctx->status; a.active = active; a.ext_target = local_target; a.token_offset = vocab_offset;
    a.pos = nullptr; a.pos_stride = 0; a.slot_stride = 0; a.thr = nullptr;
    const int S = pick_cluster(ctx, B, V_shard, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(draft_step_kernel<kBF16, false, 2>, B, S, a, st, kRingBytes)
                                       : launch_clustered(draft_step_kernel<kF32, false, 2>, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_pair_stats(svip_ctx* ctx, const void* q_logits, long q_row_stride, const void* target_logits,
                    long t_row_stride, svip_dtype dtype, int n_pairs, int V, float T, float c_bound,
                    float* out, void* stream) {
    if (!ctx || !q_logits || !target_logits || !out) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (n_pairs < 0 || V < 1 || V > 0x7fffffe0 || q_row_stride < 0 || t_row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(c_bound >= 0.f)) return SVIP_ERR_INVALID_ARG;
    const size_t esz = dtype == SVIP_BF16 ? 2 : 4;
    if (!aligned_to(target_logits, esz) || !aligned_to(q_logits, esz)) return SVIP_ERR_INVALID_ARG;
    if (n_pairs == 0) return SVIP_OK;
    if (n_pairs > ctx->max_rows) return SVIP_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float c = scale_for(T);
    const int S = pick_cluster(ctx, n_pairs, V, dtype);
    StatsArgs s;
    s.row_stride = t_row_stride; s.V = V; s.c = c; s.draft_rows = 0; s.K = 1; s.cu = nullptr;
    s.q_seq_stride = 0; s.q_pos_stride = 0; s.out_argmax = nullptr; s.status = ctx->status;
    s.out_partial = nullptr; s.idx_offset = 0;
    for (int side = 0; side < 2; ++side) {
        s.logits = side == 0 ? target_logits : q_logits;
        s.row_stride = side == 0 ? t_row_stride : q_row_stride;
        s.out_stats = side == 0 ? ctx->p_stats : ctx->q_stats;
        cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, n_pairs, S, s, st, kRingBytes)
                                           : launch_clustered(row_stats_kernel<kF32, 1>, n_pairs, S, s, st, kRingBytes);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }
    PairArgs p;
    p.t_logits = target_logits; p.t_row_stride = t_row_stride; p.q_logits = q_logits; p.q_row_stride = q_row_stride;
    p.p_stats = ctx->p_stats; p.q_stats = ctx->q_stats; p.V = V; p.c = c; p.c_bound = c_bound; p.out = out;
    p.status = ctx->status;
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(pair_stats_kernel<kBF16>, n_pairs, S, p, st, 0)
                                       : launch_clustered(pair_stats_kernel<kF32>, n_pairs, S, p, st, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_graph_begin(svip_ctx* ctx, void* stream) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    cudaError_t e = cudaSuccess;
    if (!ctx->loop_stream) {   // made now: no stream is created while a capture is open
        e = cudaStreamCreateWithFlags(&ctx->loop_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) { ctx->loop_stream = nullptr; return cuda_fail(ctx, e); }
    }
    e = cudaStreamBeginCapture(static_cast<cudaStream_t>(stream), cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->capturing = 1;
    return SVIP_OK;
}

int svip_graph_loop_begin(svip_ctx* ctx, void* stream, const int32_t* n_active, int max_iters, void** body_stream) {
    if (!ctx || !n_active || !body_stream || max_iters < 1) return SVIP_ERR_INVALID_ARG;
    if (!ctx->capturing || ctx->loop_open) return SVIP_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the iteration counter starts at zero at every replay
    cudaError_t e = cudaMemsetAsync(ctx->loop_iter, 0, sizeof(int), st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    cudaGraph_t graph = nullptr;
    const cudaGraphNode_t* deps = nullptr;
    size_t n_deps = 0;
    e = cudaStreamGetCaptureInfo(st, &status, nullptr, &graph, &deps, &n_deps);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (status != cudaStreamCaptureStatusActive || !graph) return SVIP_ERR_STATE;
    // the body runs once before the first decision (the do-while of Algorithm 1): default value 1
    cudaGraphConditionalHandle handle;
    e = cudaGraphConditionalHandleCreate(&handle, graph, 1, cudaGraphCondAssignDefault);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaGraphNodeParams params = {};
    params.type = cudaGraphNodeTypeConditional;
    params.conditional.handle = handle;
    params.conditional.type = cudaGraphCondTypeWhile;
    params.conditional.size = 1;
    cudaGraphNode_t node = nullptr;
    e = cudaGraphAddNode(&node, graph, deps, n_deps, &params);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaGraph_t body = params.conditional.phGraph_out[0];
    // from here on the graph holds a loop: if its body cannot be recorded, svip_graph_end refuses
    // to hand the graph out (a loop without a deciding kernel would never end)
    // what is recorded on `stream` from here on comes after the loop
    e = cudaStreamUpdateCaptureDependencies(st, &node, 1, cudaStreamSetCaptureDependencies);
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    e = cudaStreamBeginCaptureToGraph(ctx->loop_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    ctx->loop.handle = handle;
    ctx->loop.iter = ctx->loop_iter;
    ctx->loop.max_iters = max_iters;
    ctx->loop_n_active = n_active;
    ctx->loop_open = 1;
    ctx->loop_decided = 0;
    t_plain_launches = true;
    *body_stream = ctx->loop_stream;
    return SVIP_OK;
}

int svip_graph_loop_end(svip_ctx* ctx) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (!ctx->loop_open) return SVIP_ERR_STATE;
    cudaError_t e = cudaSuccess;
    if (!ctx->loop_decided) {   // no svip_policy_advance on the loop's counter in the body: decide here
        e = launch_ex(loop_decide_kernel, 1, 32, 0, 0, ctx->loop_stream, ctx->loop, ctx->loop_n_active);
        if (e == cudaSuccess) ctx->launches += 1;
    }
    cudaGraph_t body = nullptr;
    cudaError_t e2 = cudaStreamEndCapture(ctx->loop_stream, &body);
    ctx->loop_open = 0;
    t_plain_launches = false;
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    if (e2 != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e2); }
    return SVIP_OK;
}

int svip_graph_end(svip_ctx* ctx, void* stream, svip_graph** graph) {
    if (!ctx || !graph) return SVIP_ERR_INVALID_ARG;
    if (!ctx->capturing) return SVIP_ERR_STATE;
    // a loop whose body was left open, or whose decision kernel could not be recorded, would
    // never end at replay: such a graph is not handed out
    bool broken = ctx->loop_failed != 0;
    if (ctx->loop_open) {
        cudaGraph_t body = nullptr;
        cudaStreamEndCapture(ctx->loop_stream, &body);
        ctx->loop_open = 0;
        t_plain_launches = false;
        broken = true;
    }
    ctx->loop_failed = 0;
    ctx->capturing = 0;
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(static_cast<cudaStream_t>(stream), &g);
    if (broken) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return SVIP_ERR_STATE;
    }
    if (e != cudaSuccess || !g) return cuda_fail(ctx, e);
    cudaGraphExec_t ex = nullptr;
    e = cudaGraphInstantiate(&ex, g, 0);
    if (e != cudaSuccess) { cudaGraphDestroy(g); return cuda_fail(ctx, e); }
    svip_graph* out = new (std::nothrow) svip_graph();
    if (!out) { cudaGraphExecDestroy(ex); cudaGraphDestroy(g); return SVIP_ERR_CUDA; }
    out->exec = ex; out->graph = g;
    *graph = out;
    return SVIP_OK;
}

int svip_graph_launch(svip_graph* graph, void* stream) {
    if (!graph) return SVIP_ERR_INVALID_ARG;
    return cudaGraphLaunch(graph->exec, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SVIP_OK : SVIP_ERR_CUDA;
}

int svip_graph_destroy(svip_graph* graph) {
    if (!graph) return SVIP_ERR_INVALID_ARG;
    cudaGraphExecDestroy(graph->exec);
    cudaGraphDestroy(graph->graph);
    delete graph;
    return SVIP_OK;
}

// ------------------------------------------------------------------ verify without allocation
//
// Workspace of svip_verify_noalloc: one fixed array in the library's device image instead of
// cudaMalloc'ed memory.  Layout: [p_stats | q_stats | p_argmax | status word].  Every call on a
// device reuses it, so calls that overlap on the GPU race (see include/svip.h).

namespace {

constexpr size_t kNoAllocRows = SVIP_NOALLOC_MAX_ROWS;
constexpr size_t kNoAllocStatsBytes = kNoAllocRows * sizeof(float2);
constexpr size_t kNoAllocBytes = 2 * kNoAllocStatsBytes + kNoAllocRows * sizeof(int32_t) + 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNoAllocMaxDevices = 64;

struct NoAllocDevice {
    int ready;
    int num_sms;
    unsigned char* base;   // device address of g_noalloc_scratch on this device
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;   // the per-device set-up may be reached from several host threads

// Once per device, with that device current: the host-side name g_noalloc_scratch is not a device
// address, so ask the runtime for the address the kernels must be given.
int noalloc_setup(int device, NoAllocDevice** out) {
    if (device < 0 || device >= kNoAllocMaxDevices) return SVIP_ERR_INVALID_ARG;
    NoAllocDevice* d = &g_noalloc_dev[device];
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!d->ready) {
        int current = -1;
        if (cudaGetDevice(&current) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
        if (current != device) return SVIP_ERR_INVALID_ARG;
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return SVIP_ERR_CUDA;
        }
        if (major != 10) return SVIP_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return SVIP_ERR_CUDA;
        }
        const void* ringed[] = {
            (const void*)row_stats_kernel<kBF16, 0>, (const void*)row_stats_kernel<kBF16, 1>,
            (const void*)row_stats_kernel<kF32, 0>,  (const void*)row_stats_kernel<kF32, 1>,
            (const void*)verify_finish_kernel<kBF16>, (const void*)verify_finish_kernel<kF32>};
        for (const void* k : ringed)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes) != cudaSuccess) {
                cudaGetLastError();
                return SVIP_ERR_CUDA;
            }
        d->num_sms = sms;
        d->base = static_cast<unsigned char*>(ptr);
        d->ready = 1;
    }
    *out = d;
    return SVIP_OK;
}

}  // namespace

int svip_verify_noalloc(int device, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                        const float* q_stats, long q_seq_stride, long q_pos_stride,
                        const void* target_logits, long t_row_stride, svip_dtype dtype,
                        const int32_t* cu_rows, int B, int K, int n_target_rows, int V, float T,
                        const float* uniforms, int32_t* n_accepted, int32_t* next_token,
                        unsigned* status, void* stream) {
    if (n_target_rows > SVIP_NOALLOC_MAX_ROWS) return SVIP_ERR_WORKSPACE;
    NoAllocDevice* d = nullptr;
    int rc = noalloc_setup(device, &d);
    if (rc != SVIP_OK) return rc;
    // A context that lives on this call's stack and points into the fixed array; nothing is allocated.
    svip_ctx view = {};
    view.device = device;
    view.max_rows = SVIP_NOALLOC_MAX_ROWS;
    view.num_sms = d->num_sms;
    view.p_stats = reinterpret_cast<float2*>(d->base);
    view.q_stats = reinterpret_cast<float2*>(d->base + kNoAllocStatsBytes);
    view.p_argmax = reinterpret_cast<int32_t*>(d->base + 2 * kNoAllocStatsBytes);
    unsigned* own_status = reinterpret_cast<unsigned*>(d->base + 2 * kNoAllocStatsBytes +
                                                       kNoAllocRows * sizeof(int32_t));
    view.status = status ? status : own_status;
    // the status word must start at zero; everything else in the array is written before it is read
    if (cudaMemsetAsync(view.status, 0, sizeof(unsigned), static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return SVIP_ERR_CUDA;
    }
    return svip_verify(&view, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream);
}

}  // extern "C"
