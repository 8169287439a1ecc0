// Draft side: combining the segment partials of a row, the fine scan that finds the sampled token,
// the draft-step kernel (Algorithm 1 inner loop, Eq. 7) and the row-statistics kernel (first phase of verify).
#pragma once

#include "svip_device.cuh"
#include "svip.h"

namespace svip {

constexpr int kPolicyThreads = 256;

struct SegEntry {
    float m;
    int idx;
    float Z;
    float A;
};

// Where the entries read by combine_segments live: `Remote` reads entry s from the block that
// produced it, through distributed shared memory (the caller brackets this with cluster barriers);
// `Local` reads a block-local table that the peers have filled (SegExchange below).
struct RemoteSegments {
    cg::cluster_group& cluster;
    SegEntry* seg;
    __device__ __forceinline__ SegEntry operator()(int s) const {
        return cluster.map_shared_rank(seg, s / kWarps)[s % kWarps];
    }
};
struct LocalSegments {
    const SegEntry* all;
    __device__ __forceinline__ SegEntry operator()(int s) const { return all[s]; }
};

// Merges the nseg segment entries of a row into the row's partial and selects the segment holding
// the mass u * Z.  Warp-collective; every warp that runs it on the same entries gets the same bits.
template <int kMode, class Source>
__device__ __forceinline__ void combine_entries(const Source& src, int nseg, float c, float u, int lane,
                                                Partial& row, SegPick& pick, float abs_target = -1.f) {
    const int per = (nseg + 31) / 32;
    Partial e[kSegPerLane];
    float m = neg_inf();
#pragma unroll
    for (int k = 0; k < kSegPerLane; ++k) {
        e[k].m = neg_inf(); e[k].idx = kIntMax; e[k].Z = 0.f; e[k].A = 0.f;
        int s = lane * per + k;
        if (k < per && s < nseg) {
            SegEntry v = src(s);
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

// Reads every segment entry of the cluster through distributed shared memory (run by warp 0 of a
// block, between two cluster barriers).
template <int kMode>
__device__ __forceinline__ void combine_segments(cg::cluster_group& cluster, SegEntry* seg, int S,
                                                 float c, float u, int lane, Partial& row,
                                                 SegPick& pick, float abs_target = -1.f) {
    RemoteSegments src{cluster, seg};
    combine_entries<kMode>(src, S * kWarps, c, u, lane, row, pick, abs_target);
}

// The segment entries of a row, pushed by the warps that produced them into every block of the
// cluster (see the exchange primitives in svip_device.cuh).
struct SegExchange {
    SegEntry all[kMaxSeg];     // entry of segment s at index s
    unsigned long long bar;    // mbarrier: completes when S * kWarps entries have landed here
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// To be run by every thread of every block of the cluster before the row is streamed.
__device__ __forceinline__ void exchange_open(SegExchange& ex, int S, int tid) {
    if (S == 1) return;
    if (tid == 0) {
        const uint32_t bar = smem_addr(&ex.bar);
        mbar_init(bar, 1);
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(S * kWarps * sizeof(SegEntry)));
    }
    cluster_arrive();   // a peer pushes only after its cluster_wait(), hence after this initialisation
}

// The calling warp publishes the entry of its segment (rank * kWarps + warp) to every block.
__device__ __forceinline__ void exchange_push(SegExchange& ex, int S, int rank, int warp, int lane, const Partial& t) {
    if (S == 1) {
        if (lane == 0) { SegEntry& e = ex.all[warp]; e.m = t.m; e.idx = t.idx; e.Z = t.Z; e.A = t.A; }
        return;
    }
    cluster_wait();
    if (lane < S) {
        const uint32_t dst = map_to_rank(smem_addr(&ex.all[rank * kWarps + warp]), lane);
        const uint32_t bar = map_to_rank(smem_addr(&ex.bar), lane);
        push16(dst, bar, __float_as_uint(t.m), static_cast<uint32_t>(t.idx), __float_as_uint(t.Z), __float_as_uint(t.A));
    }
}

// Until all entries are here (S > 1; bounded): false if the wait ran out.
__device__ __forceinline__ bool exchange_wait(SegExchange& ex) {
    return mbar_wait_bounded(smem_addr(&ex.bar), 0);
}

// Fine scan of one segment by the whole block.  The functor splits into `load(vi)` (the raw 16-byte
// vectors of element-vector vi) and `weights(vi, raw, w)` (their weights), so that a thread issues all
// its loads at once and keeps them in registers.  Each thread sums a run of consecutive vectors, one
// block scan places the runs, and in every warp the lowest lane whose run crosses `target` walks its
// run again element by element; the lowest such thread of the block wins.  Returns the virtual
// element index (vector * EPV + element) of the first element whose cumulative weight exceeds
// `target`, else the last element with positive weight, else -1.  All threads return the same value.
template <int EPV, class WF>
__device__ __forceinline__ int fine_scan(const WF& wf, int v_lo, int v_hi, float prefix, float target,
                                         ScanShared& sh, int tid, int lane, int warp) {
    constexpr int kRun = 4;
    constexpr unsigned long long kNone = ~0ull;
    const int nv = v_hi - v_lo;
    const int run = min(kRun, max(1, (nv + kThreads - 1) / kThreads));
    if (tid == 0) { sh.key = kNone; sh.lastpos = -1; sh.result = -1; }
    float running = prefix;
    for (int cb = v_lo; cb < v_hi; cb += kThreads * run) {
        const int first = cb + tid * run;
        typename WF::Raw raw[kRun];
#pragma unroll
        for (int k = 0; k < kRun; ++k)
            if (k < run && first + k < v_hi) raw[k] = wf.load(first + k);
        float ls = 0.f;
        int lastv = -1;
#pragma unroll
        for (int k = 0; k < kRun; ++k) {
            if (k < run && first + k < v_hi) {
                float w[EPV];
                wf.weights(first + k, raw[k], w);
                float sv = 0.f;
#pragma unroll
                for (int j = 0; j < EPV; ++j) sv += w[j];
                if (sv > 0.f) lastv = first + k;
                ls += sv;
            }
        }
        const float inc = warp_scan_incl(ls, lane);
        __syncthreads();   // wsum is free again; the initial key is visible
        if (lane == 31) sh.wsum[warp] = inc;
        __syncthreads();
        float before = 0.f, total = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float sw = sh.wsum[w];
            if (w < warp) before += sw;
            total += sw;
        }
        const float lo = running + (before + (inc - ls));
        const unsigned crossing = __ballot_sync(0xffffffffu, ls > 0.f && lo + ls > target);
        if (crossing && lane == __ffs(crossing) - 1) {
            float cum = lo;
            int res = -1, last = -1;
#pragma unroll
            for (int k = 0; k < kRun; ++k) {
                if (k < run && first + k < v_hi) {
                    float w[EPV];
                    wf.weights(first + k, raw[k], w);
#pragma unroll
                    for (int j = 0; j < EPV; ++j) {
                        cum += w[j];
                        if (w[j] > 0.f) {
                            last = (first + k) * EPV + j;
                            if (cum > target && res < 0) res = last;
                        }
                    }
                }
            }
            atomicMin(&sh.key, (static_cast<unsigned long long>(tid) << 32) |
                                   static_cast<unsigned>(res >= 0 ? res : last));
        }
        const int lv = __reduce_max_sync(0xffffffffu, lastv);
        if (lane == 0 && lv >= 0) atomicMax(&sh.lastpos, lv);
        __syncthreads();
        const unsigned long long key = sh.key;
        if (key != kNone) return static_cast<int>(static_cast<unsigned>(key & 0xffffffffull));
        running += total;
    }
    // rounding left nothing above the target: the last element with weight
    const int lv = sh.lastpos;
    if (lv < 0) return -1;
    if (tid == 0) {
        float w[EPV];
        wf.weights(lv, wf.load(lv), w);
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
    typedef uint4 Raw;
    __device__ __forceinline__ Raw load(int vi) const { return ld_vec(g.base + vi); }
    __device__ __forceinline__ void weights(int vi, const Raw& raw, float (&w)[ElemTraits<DT>::kEPV]) const {
        constexpr int EPV = ElemTraits<DT>::kEPV;
        float x[EPV];
        unpack_masked<DT>(raw, vi, g, x);
#pragma unroll
        for (int j = 0; j < EPV; ++j)
            w[j] = x[j] >= thr ? ex2_approx(fmaxf(__fmaf_rn(x[j], c, -M), kArgFloor)) : 0.f;
    }
};

struct RowShared {
    Partial row;
    SegPick pick;
};

// The draft step of one row by the cluster that shares it: stream the row (Z, A, maximum), push the
// segment partials to every block of the cluster, combine them (every block the same bits), write
// entropy / stop flag / normalisers, and let the block that holds the sampled mass find the token.
// `g` describes the row, `thr` is the truncation threshold when kThr.  No block reads a peer's shared
// memory, and a block leaves only after every entry aimed at it has landed.
template <int DT, bool kGreedy, bool kPos, bool kThr>
__device__ __forceinline__ void draft_row(const DraftArgs& a, cg::cluster_group& cluster, int S, int rank, int row,
                                          int tid, const RowGeom g, const uint32_t slot0, const long p, const float thr) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    const int lane = tid & 31, warp = tid >> 5;
    __shared__ SegExchange ex;
    __shared__ ScanShared scan;
    __shared__ RowShared res;
    exchange_open(ex, S, tid);
    float u = 0.f, ext = -1.f;
    if (!kGreedy && warp == 0) {   // fetched now, used after the stream
        if (a.ext_target) ext = fmaxf(__ldg(a.ext_target + row), 0.f);
        else u = __ldg(a.uniforms + (row + p * a.slot_stride));
    }
    Partial t = reduce_segment<DT, 2, kGreedy, kThr>(g, rank * kWarps + warp, a.c, lane, slot0, thr);
    exchange_push(ex, S, rank, warp, lane, t);
    if (S == 1) __syncthreads();
    if (warp == 0) {
        if (S > 1 && !exchange_wait(ex) && lane == 0) atomicOr(a.status, SVIP_STATUS_WAIT_TIMEOUT);
        Partial r; SegPick pk;
        LocalSegments src{ex.all};
        combine_entries<2>(src, S * kWarps, a.c, u, lane, r, pk, ext);
        if (lane == 0) { res.row = r; res.pick = pk; }
    }
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
}

// kBlocks is the number of blocks the register budget must leave room for on one SM: 2 for
// launches that fit the GPU in one wave (latency matters, registers are free), 3 for launches of
// many waves, where a third resident block streams on while another one is in its epilogue.
// kPos compiles the position-indexed form (svip_draft_step_at) in, kThr the truncated form
// (svip_draft_step_filtered).
template <int DT, bool kGreedy, int kBlocks, bool kPos = false, bool kThr = false>
__global__ void __launch_bounds__(kThreads, kBlocks) draft_step_kernel(DraftArgs a) {
    extern __shared__ uint4 ring[];
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int row = blockIdx.x / S;
    const int tid = threadIdx.x;

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
    const float thr = kThr ? a.thr[row] : neg_inf();
    draft_row<DT, kGreedy, kPos, kThr>(a, cluster, S, rank, row, tid, g, slot0, p, thr);
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

}  // namespace svip
