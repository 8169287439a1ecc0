// Truncation threshold of a logits row (top-k and nucleus / top-p).
//
// The kept set of a row is {i : l_i >= tau}: tau_k is the k-th largest logit, and inside that set
// tau is the largest logit value v for which the mass of {l_i >= v} reaches top_p of the mass of
// {l_i >= tau_k}; tokens tied with the last kept one are all kept.  The paper applies its length
// policy on top of samplers that truncate but does not define the truncation; these are the
// published definitions (top-k, nucleus sampling) read with a threshold so that the result does not
// depend on the order of equal logits.
//
// One cluster per row.  Top-k with a small k takes two passes and a handful of candidates (see
// candidate_path below).  Otherwise the value is found by a radix descent over an order-preserving integer
// image of the logits, 8 bits per pass: every pass streams the row once (cp.async ring, as the other
// kernels), histograms the digit of the elements that match the digits already fixed (counts, and
// for the nucleus the masses 2^(l*c - M) in 2^-40 fixed point, so that every sum is an integer and
// the result is the same whatever the order of the additions), the blocks add their histograms up
// through distributed shared memory, and every block takes the same decision from the same sums.
// bf16 rows need two passes per descent, fp32 rows four.
#pragma once

#include "svip_device.cuh"
#include "svip_draft.cuh"

namespace svip {

constexpr int kHistCopies = 8;           // interleaved copies of the histogram: lane l adds into copy l % 8, so
                                         // lanes that meet in one bin mostly hit different words and banks
constexpr float kMassScale = 1099511627776.0f;   // 2^40
constexpr int kCandPerBlock = 1024;      // candidate keys a block may collect
constexpr int kPoolCap = 4096;           // candidate keys of the whole cluster (lives in the histogram copies)
constexpr int kPoolCapDraft = 2048;      // the same when their indices are kept too (draft form)
constexpr int kSmallPool = 256;          // up to this many candidates are ranked by plain counting

struct ThresholdArgs {
    const void* logits;
    long row_stride;
    int V;
    float c;        // log2(e) / T
    int top_k;      // 1 .. V-1, or 0 when off
    float top_p;    // (0, 1), or >= 1 when off
    float* thr;     // [rows] out: tau as a logit value (-inf: nothing is dropped)
    float2* stats;  // [rows] out or NULL: (largest logit, mass of the kept set relative to it)
    // draft form (kDraft): the whole truncated draft step where the candidates allow it
    const float* uniforms;   // [rows]
    const uint8_t* active;   // NULL, or rows with 0 are skipped
    float thresh;            // h of the stop test
    int32_t* token;          // [rows] out
    float* entropy;          // [rows] out
    uint8_t* stop;           // [rows] out
    unsigned* status;        // device status word
    int sample_den;          // candidate path: the first bound comes from 1/sample_den of every warp segment (1: all)
};

// Monotone image of a float: a < b  <=>  key(a) < key(b).  NaN counts as -inf.
__device__ __forceinline__ uint32_t order_key(float x) {
    x = fmaxf(x, neg_inf());        // NaN -> -inf (the maximum of a NaN and a number is the number)
    x = x + 0.f;                    // -0 -> +0: the two zeros are one value
    const uint32_t u = __float_as_uint(x);
    return u ^ (static_cast<uint32_t>(static_cast<int32_t>(u) >> 31) | 0x80000000u);
}

__device__ __forceinline__ float key_value(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Streams segment `seg` of the row with the calling warp and hands every vector to f(x, vi), with
// the elements outside the row set to -inf.  den > 1: only the first 1/den of the segment (rounded up).
template <int DT, class F>
__device__ __forceinline__ void stream_segment(const RowGeom& g, int seg, int lane, uint32_t slot0, F&& f, int den = 1) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    constexpr uint32_t kSlotStride = kThreads * 16;
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    if (den > 1) v_hi = min(v_hi, v_lo + (v_hi - v_lo + den - 1) / den);
    const int vi0 = v_lo + lane;
    const int n = v_hi > vi0 ? (v_hi - vi0 + 31) >> 5 : 0;
    const uint4* src = g.base + vi0;
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
        if (s < n) cp_async16(slot0 + s * kSlotStride, src + 32 * s);
        cp_async_commit();
    }
    for (int it = 0; it < n; ++it) {
        cp_async_wait<kStages - 1>();
        const uint32_t slot = slot0 + (it & (kStages - 1)) * kSlotStride;
        const uint4 raw = lds128(slot);
        if (it + kStages < n) cp_async16(slot, src + 32 * (it + kStages));
        cp_async_commit();
        float x[EPV];
        unpack_masked<DT>(raw, vi0 + 32 * it, g, x);
        f(x, vi0 + 32 * it);
    }
    cp_async_wait<0>();
}

struct SelectShared {
    uint32_t priv[3][256][kHistCopies];   // count, mass low word, mass high word; per digit, per copy
    uint32_t blk_cnt[256];                // this block's histogram, read by the peers
    unsigned long long blk_mass[256];
    uint32_t tot_cnt[256];                // the cluster's histogram
    unsigned long long tot_mass[256];
    float blk_max;                        // this block's largest logit
    unsigned long long blk_above;         // this block's mass of the elements >= tau_k
    float warp_max[kWarps];
    unsigned long long warp_above[kWarps];
    // candidate path (top-k with a small k)
    uint32_t lane_key[kThreads];          // key of the largest logit each thread saw
    alignas(8) uint32_t cand[kCandPerBlock];   // keys of this block's elements >= the lower bound
    uint32_t cand_idx[kCandPerBlock];     // draft form: their positions in the row
    uint32_t cand_n;                      // how many there are (may exceed the capacity: then the path is left)
    uint32_t sel, sel2;                   // results of selections by counting
    uint32_t peer_n[kMaxCluster];         // candidates held by each block of the cluster
    // decision of a pass (written by warp 0)
    int bin;
    uint32_t cnt_above;
    unsigned long long mass_above;
    unsigned long long mass_total;
    unsigned long long mass_bin;
};

__device__ __forceinline__ unsigned long long shfl_up_u64(unsigned long long v, int o) {
    uint32_t lo = __shfl_up_sync(0xffffffffu, static_cast<uint32_t>(v), o);
    uint32_t hi = __shfl_up_sync(0xffffffffu, static_cast<uint32_t>(v >> 32), o);
    return (static_cast<unsigned long long>(hi) << 32) | lo;
}

// One pass: histogram of digit (key >> shift) & 255 over the elements whose higher digits equal
// those of `prefix` (all elements when first).  kMass adds the masses; kMax also finds the largest
// logit; `key_k` (with kAbove) sums the mass of the elements with key >= key_k.  On return every
// block of the cluster holds the cluster-wide histogram in sh.tot_*.
template <int DT, bool kMass, bool kMax, bool kAbove>
__device__ __forceinline__ void histogram_pass(cg::cluster_group& cluster, const RowGeom& g, int S, int rank,
                                               int tid, uint32_t slot0, uint32_t prefix, int shift, bool first,
                                               float c, float M, uint32_t key_k, SelectShared& sh,
                                               float& row_max, unsigned long long& above) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    const int lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < kHistCopies * 3 * 256; i += kThreads) (&sh.priv[0][0][0])[i] = 0;
    __syncthreads();
    uint32_t* h_cnt = &sh.priv[0][0][lane % kHistCopies];
    uint32_t* h_lo = &sh.priv[1][0][lane % kHistCopies];
    uint32_t* h_hi = &sh.priv[2][0][lane % kHistCopies];
    float mx = neg_inf();
    unsigned long long ab = 0;
    const uint32_t want = first ? 0u : (prefix >> (shift + 8));
    stream_segment<DT>(g, rank * kWarps + warp, lane, slot0, [&](const float (&x)[EPV], int) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            const uint32_t key = order_key(x[j]);
            if (kMax) mx = fmaxf(mx, x[j]);
            unsigned long long wq = 0;
            if (kMass) {
                const float w = ex2_approx(fmaxf(__fmaf_rn(x[j], c, -M), kArgFloor));
                wq = __float2ull_rz(w * kMassScale);
                if (kAbove && key >= key_k) ab += wq;
            }
            // the nucleus descent is decided by the masses alone, the top-k descent by the counts
            if ((first || (key >> (shift + 8)) == want) && (!kMass || wq)) {
                const uint32_t bin = ((key >> shift) & 255u) * kHistCopies;
                if (!kMass) {
                    atomicAdd(h_cnt + bin, 1u);
                } else {
                    const uint32_t lo = static_cast<uint32_t>(wq);
                    const uint32_t old = atomicAdd(h_lo + bin, lo);
                    const uint32_t carry = (old + lo < old) ? 1u : 0u;
                    const uint32_t hi = static_cast<uint32_t>(wq >> 32) + carry;
                    if (hi) atomicAdd(h_hi + bin, hi);
                }
            }
        }
    });
    if (kMax) {
        mx = warp_max(mx);
        if (lane == 0) sh.warp_max[warp] = mx;
    }
    if (kAbove) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            uint32_t lo = __shfl_xor_sync(0xffffffffu, static_cast<uint32_t>(ab), o);
            uint32_t hi = __shfl_xor_sync(0xffffffffu, static_cast<uint32_t>(ab >> 32), o);
            ab += (static_cast<unsigned long long>(hi) << 32) | lo;
        }
        if (lane == 0) sh.warp_above[warp] = ab;
    }
    __syncthreads();
    if (tid < 256) {
        uint32_t cn = 0;
        unsigned long long ms = 0;
#pragma unroll
        for (int k = 0; k < kHistCopies; ++k) {
            cn += sh.priv[0][tid][k];
            if (kMass) ms += (static_cast<unsigned long long>(sh.priv[2][tid][k]) << 32) + sh.priv[1][tid][k];
        }
        sh.blk_cnt[tid] = cn;
        sh.blk_mass[tid] = ms;
    }
    if (tid == 0) {
        float m = neg_inf();
        unsigned long long s = 0;
        for (int w = 0; w < kWarps; ++w) {
            if (kMax) m = fmaxf(m, sh.warp_max[w]);
            if (kAbove) s += sh.warp_above[w];
        }
        sh.blk_max = m;
        sh.blk_above = s;
    }
    cluster.sync();
    if (tid < 256) {
        uint32_t cn = 0;
        unsigned long long ms = 0;
        for (int r = 0; r < S; ++r) {
            const SelectShared* peer = cluster.map_shared_rank(&sh, r);
            cn += peer->blk_cnt[tid];
            if (kMass) ms += peer->blk_mass[tid];
        }
        sh.tot_cnt[tid] = cn;
        sh.tot_mass[tid] = ms;
    }
    if (kMax || kAbove) {
        float m = neg_inf();
        unsigned long long s = 0;
        for (int r = 0; r < S; ++r) {
            const SelectShared* peer = cluster.map_shared_rank(&sh, r);
            if (kMax) m = fmaxf(m, peer->blk_max);
            if (kAbove) s += peer->blk_above;
        }
        if (kMax) row_max = m;
        if (kAbove) above = s;
    }
    cluster.sync();   // every peer has read this block's histogram; tot_* is visible block-wide
}

// Warp 0: walks the cluster histogram from the highest digit down and finds the digit at which
// the running count reaches `k_rem` (kByMass false) or the running mass reaches `p_rem`.
template <bool kByMass>
__device__ __forceinline__ void decide(SelectShared& sh, int lane, uint32_t k_rem, unsigned long long p_rem) {
    // lane l owns the digits 255 - 8l ... 248 - 8l, highest first
    uint32_t cn[8];
    unsigned long long ms[8];
    uint32_t csum = 0;
    unsigned long long msum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int bin = 255 - 8 * lane - j;
        cn[j] = sh.tot_cnt[bin];
        ms[j] = sh.tot_mass[bin];
        csum += cn[j];
        msum += ms[j];
    }
    uint32_t cinc = csum;
    unsigned long long minc = msum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t cu = __shfl_up_sync(0xffffffffu, cinc, o);
        const unsigned long long mu = shfl_up_u64(minc, o);
        if (lane >= o) { cinc += cu; minc += mu; }
    }
    uint32_t cbefore = cinc - csum;              // digits above this lane's
    unsigned long long mbefore = minc - msum;
    int hit = -1;
    uint32_t c_at = 0;
    unsigned long long m_at = 0, m_bin = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const bool reached = kByMass ? (mbefore + ms[j] >= p_rem) : (cbefore + cn[j] >= k_rem);
        if (hit < 0 && reached && (kByMass ? ms[j] > 0 : cn[j] > 0)) {
            hit = 255 - 8 * lane - j;
            c_at = cbefore;
            m_at = mbefore;
            m_bin = ms[j];
        }
        cbefore += cn[j];
        mbefore += ms[j];
    }
    const unsigned who = __ballot_sync(0xffffffffu, hit >= 0);
    const unsigned long long total = __shfl_sync(0xffffffffu, static_cast<uint32_t>(minc), 31) |
        (static_cast<unsigned long long>(__shfl_sync(0xffffffffu, static_cast<uint32_t>(minc >> 32), 31)) << 32);
    if (who == 0) {
        // nothing reaches the target (an empty histogram): stay at the lowest digit
        if (lane == 0) { sh.bin = 0; sh.cnt_above = 0; sh.mass_above = 0; sh.mass_total = total; sh.mass_bin = 0; }
    } else if (lane == __ffs(who) - 1) {
        sh.bin = hit; sh.cnt_above = c_at; sh.mass_above = m_at; sh.mass_total = total; sh.mass_bin = m_bin;
    }
}

// Sum of one 64-bit integer per thread over the block (every thread gets it).  Two barriers.
__device__ __forceinline__ unsigned long long block_sum_u64(SelectShared& sh, unsigned long long v, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        uint32_t lo = __shfl_xor_sync(0xffffffffu, static_cast<uint32_t>(v), o);
        uint32_t hi = __shfl_xor_sync(0xffffffffu, static_cast<uint32_t>(v >> 32), o);
        v += (static_cast<unsigned long long>(hi) << 32) | lo;
    }
    __syncthreads();   // warp_above may still be read from an earlier use
    if (lane == 0) sh.warp_above[warp] = v;
    __syncthreads();
    v = 0;
    for (int w = 0; w < kWarps; ++w) v += sh.warp_above[w];
    return v;
}

// What the statistics output holds for a row: (m, Z~) in the convention of the draft step's row_stats.
__device__ __forceinline__ float2 kept_stats(float row_max, unsigned long long kept_mass, bool finite) {
    return make_float2(row_max, finite ? static_cast<float>(static_cast<double>(kept_mass) / 1099511627776.0) : 0.f);
}

__device__ __forceinline__ unsigned long long mass_of_key(uint32_t key, float c, float M) {
    const float w = ex2_approx(fmaxf(__fmaf_rn(key_value(key), c, -M), kArgFloor));
    return __float2ull_rz(w * kMassScale);
}

// Radix descent over `n` keys held in shared memory, the same in every block of the cluster, so
// no exchange is needed: the k_rem-th largest key (by counts), or the key at which the running mass
// from the top reaches p_rem.  Block-collective.
template <int kLevels, bool kByMass>
__device__ __forceinline__ uint32_t pool_select(SelectShared& sh, const uint32_t* pool, int n, uint32_t k_rem,
                                                unsigned long long p_rem, float c, float M, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t prefix = 0;
    for (int level = 0; level < kLevels; ++level) {
        const int shift = 24 - 8 * level;
        if (tid < 256) { sh.tot_cnt[tid] = 0; sh.tot_mass[tid] = 0; }
        __syncthreads();
        for (int i = tid; i < n; i += kThreads) {
            const uint32_t key = pool[i];
            if (level == 0 || (key >> (shift + 8)) == (prefix >> (shift + 8))) {
                const uint32_t bin = (key >> shift) & 255u;
                if (!kByMass) {
                    atomicAdd(&sh.tot_cnt[bin], 1u);
                } else {
                    const unsigned long long wq = mass_of_key(key, c, M);
                    if (wq) atomicAdd(&sh.tot_mass[bin], wq);
                }
            }
        }
        __syncthreads();
        if (warp == 0) decide<kByMass>(sh, lane, k_rem, p_rem);
        __syncthreads();
        prefix |= static_cast<uint32_t>(sh.bin) << shift;
        k_rem -= sh.cnt_above;
        p_rem -= sh.mass_above;
        __syncthreads();
    }
    if (kLevels == 2 && !(prefix & 0x80000000u)) prefix |= 0xffffu;
    return prefix;
}

// Sum over the warp of per-lane masses below 2^48 (a lane adds up at most 8 masses of about 2^40):
// two 32-bit integer reductions over a 24-bit and a 24-bit limb, neither of which can overflow.
__device__ __forceinline__ unsigned long long warp_sum_mass(unsigned long long v) {
    const uint32_t lo = __reduce_add_sync(0xffffffffu, static_cast<uint32_t>(v) & 0xffffffu);
    const uint32_t hi = __reduce_add_sync(0xffffffffu, static_cast<uint32_t>(v >> 24));
    return (static_cast<unsigned long long>(hi) << 24) + lo;
}

// Everything after the candidates are gathered, for a small set (n <= kSmallPool), by plain counting,
// one warp per candidate (the lanes share the other candidates) and two block barriers: the k-th
// largest key has fewer than k keys above it and at least k at or above it; the nucleus cut has less
// than the target mass strictly above it and at least the target at or above it; the sampled token
// is the kept candidate whose running mass in index order first exceeds u * total.  Masses are the
// 2^-40 fixed-point integers used everywhere in this file, so nothing depends on the order of the
// candidates.  Returns the key of tau; `drafted` (kDraft; the same in every block) tells whether
// block 0 has written token, entropy and stop flag.
template <bool kDraft>
__device__ __forceinline__ uint32_t small_finish(SelectShared& sh, const uint32_t* pool, const uint32_t* pool_idx,
                                                 int n, const ThresholdArgs& a, bool use_p, int row, int rank, int tid,
                                                 bool& drafted) {
    const int lane = tid & 31, warp = tid >> 5;
    // this block's own candidates have been copied by every peer: their place holds the masses now
    unsigned long long* wq = reinterpret_cast<unsigned long long*>(sh.cand);
    if (tid == 0) { sh.sel = 0; sh.sel2 = 0; }
    uint32_t top = 0;
    for (int j = lane; j < n; j += 32) top = max(top, pool[j]);
    top = __reduce_max_sync(0xffffffffu, top);
    const float row_max = key_value(top);          // the largest candidate is the largest logit of the row
    const bool finite = fabsf(row_max) <= kMaxLogit;
    const float M = finite ? __fmul_rn(row_max, a.c) : 0.f;
    __syncthreads();
    const uint32_t k = static_cast<uint32_t>(a.top_k);
    for (int i = warp; i < n; i += kWarps) {
        const uint32_t key = pool[i];
        uint32_t gt = 0, ge = 0;
        for (int j = lane; j < n; j += 32) {
            const uint32_t kj = pool[j];
            gt += kj > key ? 1u : 0u;
            ge += kj >= key ? 1u : 0u;
        }
        gt = __reduce_add_sync(0xffffffffu, gt);
        ge = __reduce_add_sync(0xffffffffu, ge);
        if (lane == 0) {
            if (gt < k && k <= ge) sh.sel = key;   // every candidate that qualifies holds the same key
            wq[i] = mass_of_key(key, a.c, M);
        }
    }
    __syncthreads();
    const uint32_t key_k = sh.sel;
    uint32_t key_t = key_k;
    if (use_p && finite) {
        unsigned long long zk = 0;
        for (int j = lane; j < n; j += 32)
            if (pool[j] >= key_k) zk += wq[j];
        zk = warp_sum_mass(zk);
        if (zk > 0) {
            const double want = ceil(static_cast<double>(a.top_p) * static_cast<double>(zk));
            unsigned long long p_rem = static_cast<unsigned long long>(want);
            if (p_rem < 1) p_rem = 1;
            if (p_rem > zk) p_rem = zk;
            for (int i = warp; i < n; i += kWarps) {
                const uint32_t key = pool[i];
                if (key < key_k) continue;          // warp-uniform
                unsigned long long mgt = 0, mge = 0;
                for (int j = lane; j < n; j += 32) {
                    const uint32_t kj = pool[j];
                    const unsigned long long w = wq[j];
                    if (kj > key) mgt += w;
                    if (kj >= key) mge += w;
                }
                mgt = warp_sum_mass(mgt);
                mge = warp_sum_mass(mge);
                if (lane == 0 && mgt < p_rem && p_rem <= mge) sh.sel2 = key;
            }
        }
        __syncthreads();
        if (sh.sel2 > key_t) key_t = sh.sel2;
    }
    drafted = false;
    if (a.stats || kDraft) {
        unsigned long long zt = 0;
        for (int j = lane; j < n; j += 32)
            if (pool[j] >= key_t) zt += wq[j];
        zt = warp_sum_mass(zt);
        if (a.stats && rank == 0 && tid == 0) a.stats[row] = kept_stats(row_max, zt, finite);
        drafted = kDraft && finite && zt > 0;   // the same in every block of the cluster
        if (drafted && rank == 0) {
            long long term = 0;
            if (tid < n && pool[tid] >= key_t) {
                const float arg = fmaxf(__fmaf_rn(key_value(pool[tid]), a.c, -M), kArgFloor);
                term = __float2ll_rz(ex2_approx(arg) * arg * kMassScale);
            }
            const long long aq = static_cast<long long>(block_sum_u64(sh, static_cast<unsigned long long>(term), tid));
            const float u = a.uniforms[row];
            const unsigned long long target = static_cast<unsigned long long>(static_cast<double>(u) * static_cast<double>(zt));
            for (int i = warp; i < n; i += kWarps) {
                if (pool[i] < key_t) continue;      // warp-uniform
                const uint32_t at = pool_idx[i];
                unsigned long long cum = 0;
                for (int j = lane; j < n; j += 32)
                    if (pool[j] >= key_t && pool_idx[j] <= at) cum += wq[j];
                cum = warp_sum_mass(cum);
                if (lane == 0 && cum > target && cum - wq[i] <= target) {   // exactly one kept candidate
                    const float Z = static_cast<float>(static_cast<double>(zt) / 1099511627776.0);
                    const float A = static_cast<float>(static_cast<double>(aq) / 1099511627776.0);
                    const float H = fmaxf(kLn2 * (log2f(Z) - A / Z), 0.f);
                    a.token[row] = static_cast<int32_t>(at);
                    a.entropy[row] = H;
                    a.stop[row] = __fsqrt_rn(H) > a.thresh ? 1 : 0;
                }
            }
        }
    }
    return key_t;
}

// The truncated draft step from the candidates alone (block-collective, run by one block): the kept
// tokens are the candidates with key >= key_t.  Their masses are 2^-40 fixed point, so the
// normaliser, the entropy sums and the running sums of the inverse CDF are integers and do not
// depend on the order in which the candidates were collected.  The kept candidates are put in
// index order (`scratch`, 24 KB of shared memory no longer used for streaming) by counting, for
// each, the kept candidates before it; the token is the first whose running mass exceeds
// u * total.  Returns false, having written nothing, for a row without finite mass.
__device__ __forceinline__ bool draft_from_candidates(SelectShared& sh, const uint32_t* pool, const uint32_t* pool_idx,
                                                      int total, uint32_t key_t, float row_max, float M, bool finite,
                                                      const ThresholdArgs& a, int row, void* scratch, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
    unsigned long long* wq_sorted = static_cast<unsigned long long*>(scratch);
    uint32_t* idx_sorted = reinterpret_cast<uint32_t*>(wq_sorted + kPoolCapDraft);
    unsigned long long zq = 0, nk = 0;
    long long aq = 0;
    for (int i = tid; i < total; i += kThreads) {
        const uint32_t key = pool[i];
        if (key < key_t) continue;
        const float arg = fmaxf(__fmaf_rn(key_value(key), a.c, -M), kArgFloor);
        const float w = ex2_approx(arg);
        const unsigned long long wq = __float2ull_rz(w * kMassScale);
        zq += wq;
        aq += __float2ll_rz(w * arg * kMassScale);
        nk += 1;
        const uint32_t mine = pool_idx[i];
        int before = 0;
        for (int j = 0; j < total; ++j) before += (pool[j] >= key_t && pool_idx[j] < mine) ? 1 : 0;
        wq_sorted[before] = wq;
        idx_sorted[before] = mine;
    }
    zq = block_sum_u64(sh, zq, tid);
    aq = static_cast<long long>(block_sum_u64(sh, static_cast<unsigned long long>(aq), tid));
    nk = block_sum_u64(sh, nk, tid);
    if (!finite || zq == 0 || nk == 0) return false;
    if (warp == 0) {
        const int n = static_cast<int>(nk);
        const float u = a.uniforms[row];
        const unsigned long long target = static_cast<unsigned long long>(static_cast<double>(u) * static_cast<double>(zq));
        const int per = (n + 31) / 32;
        const int lo = min(lane * per, n), hi = min(lo + per, n);
        unsigned long long sum = 0;
        for (int i = lo; i < hi; ++i) sum += wq_sorted[i];
        unsigned long long incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = shfl_up_u64(incl, o);
            if (lane >= o) incl += up;
        }
        unsigned long long cum = incl - sum;
        int pos = kIntMax;
        for (int i = lo; i < hi; ++i) {
            cum += wq_sorted[i];
            if (cum > target && pos == kIntMax) pos = i;
        }
        pos = warp_min_int(pos);
        if (pos == kIntMax) pos = n - 1;
        if (lane == 0) {
            const float Z = static_cast<float>(static_cast<double>(zq) / 1099511627776.0);
            const float A = static_cast<float>(static_cast<double>(aq) / 1099511627776.0);
            const float H = fmaxf(kLn2 * (log2f(Z) - A / Z), 0.f);
            a.token[row] = static_cast<int32_t>(idx_sorted[pos]);
            a.entropy[row] = H;
            a.stop[row] = __fsqrt_rn(H) > a.thresh ? 1 : 0;
            if (a.stats) a.stats[row] = make_float2(row_max, Z);
        }
    }
    return true;
}

// Top-k (and the nucleus inside it) for a small k, in two passes over the row.  Pass 1 leaves the
// largest logit of every thread; the k-th largest of these S * 512 values is a lower bound t0 of
// tau_k (they are k distinct elements of the row).  Pass 2 collects every element >= t0 -- a few more
// than k when k is small against the number of threads.  tau_k, the mass of the top-k set and the
// nucleus cut then come from these candidates alone, which every block of the cluster holds in
// full.  Returns false (for the whole cluster alike) when the candidates do not fit; nothing has
// been written then and the caller takes the radix descent over the full row.
// kDraft also keeps the positions of the candidates and lets block 0 finish the whole draft step from
// them (`drafted`, the same in every block); `scratch` is the streaming ring, free by then.
// sample_den > 1: pass 1 reads only the first 1/sample_den of every warp segment.  The k-th largest of the
// thread maxima of that part is still k distinct elements of the row, hence still a lower bound of tau_k,
// only a looser one (about sample_den * k candidates instead of k); pass 2 then finds that part in L2, so the
// row crosses HBM 1 + 1 / sample_den times instead of twice.  *overflow tells a set that did not fit from a set
// that is too small.
template <int DT, bool kDraft>
__device__ __forceinline__ bool candidate_path(cg::cluster_group& cluster, const RowGeom& g, int S, int rank, int tid,
                                               uint32_t slot0, const ThresholdArgs& a, bool use_p, SelectShared& sh,
                                               uint32_t& key_out, void* scratch, bool& drafted, int sample_den,
                                               bool* overflow) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    constexpr int kLevels = DT == kBF16 ? 2 : 4;
    constexpr int kCap = kDraft ? kPoolCapDraft : kPoolCap;
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t* pool = &sh.priv[0][0][0];
    uint32_t* pool_idx = pool + kPoolCapDraft;
    static_assert(sizeof(sh.priv) >= kPoolCap * sizeof(uint32_t), "the pool lives in the histogram copies");
    drafted = false;
    // pass 1: the largest logit of every thread (fmaxf skips NaN); threads without elements keep key 0
    float best = neg_inf();
    bool any = false;
    stream_segment<DT>(g, rank * kWarps + warp, lane, slot0, [&](const float (&x)[EPV], int) {
        any = true;
#pragma unroll
        for (int j = 0; j < EPV; ++j) best = fmaxf(best, x[j]);
    }, sample_den);
    sh.lane_key[tid] = any ? order_key(best) : 0u;
    if (tid == 0) sh.cand_n = 0;
    cluster.sync();
    const int n_lane = S * kThreads;
    for (int r = 0; r < S; ++r) pool[r * kThreads + tid] = cluster.map_shared_rank(&sh, r)->lane_key[tid];
    __syncthreads();
    // only a lower bound is needed: two digits of the k-th largest maximum, the rest taken as zero
    const uint32_t t0 = pool_select<2, false>(sh, pool, n_lane, static_cast<uint32_t>(a.top_k), 0ull, 0.f, 0.f, tid) &
                        0xffff0000u;
    // pass 2: every element at or above the lower bound.  Comparing the logits is comparing the keys,
    // except for NaN, which counts as -inf and so belongs to the candidates only when the bound is that low.
    const float t0v = t0 > 0x007fffffu ? key_value(t0) : neg_inf();   // at or below the key of -inf: no bound
    const bool lowest = !(t0v > neg_inf());
    stream_segment<DT>(g, rank * kWarps + warp, lane, slot0, [&](const float (&x)[EPV], int vi) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            if (x[j] >= t0v || (lowest && !(x[j] == x[j]))) {
                const uint32_t pos = atomicAdd(&sh.cand_n, 1u);
                if (pos < kCandPerBlock) {
                    sh.cand[pos] = order_key(x[j]);
                    if (kDraft) sh.cand_idx[pos] = static_cast<uint32_t>(vi * EPV + j - g.pre);
                }
            }
        }
    });
    cluster.sync();     // every block's candidates are complete (and nobody still reads lane_key)
    if (tid < S) sh.peer_n[tid] = cluster.map_shared_rank(&sh, tid)->cand_n;   // one remote read each, side by side
    __syncthreads();
    int total = 0;
    bool fits = true;
    for (int r = 0; r < S; ++r) {
        const uint32_t nr = sh.peer_n[r];
        if (nr > kCandPerBlock) fits = false;
        total += static_cast<int>(min(nr, static_cast<uint32_t>(kCandPerBlock)));
    }
    if (total > kCap) fits = false;
    if (fits) {
        // candidate t of the cluster is candidate t - (candidates of the blocks before) of its block
        for (int t = tid; t < total; t += kThreads) {
            int r = 0, at = t;
            while (at >= static_cast<int>(sh.peer_n[r])) { at -= static_cast<int>(sh.peer_n[r]); ++r; }
            const SelectShared* peer = cluster.map_shared_rank(&sh, r);
            pool[t] = peer->cand[at];
            if (kDraft) pool_idx[t] = peer->cand_idx[at];
        }
    }
    cluster.sync();     // the peers have read this block's candidates
    *overflow = !fits;
    if (!fits || total < a.top_k) return false;
    const int row = static_cast<int>(blockIdx.x / S);
    if (total <= kSmallPool) {
        key_out = small_finish<kDraft>(sh, pool, pool_idx, total, a, use_p, row, rank, tid, drafted);
        return true;
    }
    uint32_t key_k = pool_select<kLevels, false>(sh, pool, total, static_cast<uint32_t>(a.top_k), 0ull, 0.f, 0.f, tid);
    uint32_t key_t = key_k;
    float row_max = neg_inf();
    bool finite = false;
    float M = 0.f;
    if (use_p || a.stats || kDraft) {
        // the largest candidate is the largest logit of the row
        uint32_t top = 0;
        for (int i = tid; i < total; i += kThreads) top = max(top, pool[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) top = max(top, __shfl_xor_sync(0xffffffffu, top, o));
        if (lane == 0) sh.warp_max[warp] = __uint_as_float(top);
        __syncthreads();
        top = 0;
        for (int w = 0; w < kWarps; ++w) top = max(top, __float_as_uint(sh.warp_max[w]));
        row_max = key_value(top);
        finite = fabsf(row_max) <= kMaxLogit;
        M = finite ? __fmul_rn(row_max, a.c) : 0.f;
    }
    if (use_p) {
        unsigned long long zk = 0;
        for (int i = tid; i < total; i += kThreads)
            if (pool[i] >= key_k) zk += mass_of_key(pool[i], a.c, M);
        zk = block_sum_u64(sh, zk, tid);
        if (finite && zk > 0) {
            const double want = ceil(static_cast<double>(a.top_p) * static_cast<double>(zk));
            unsigned long long p_rem = static_cast<unsigned long long>(want);
            if (p_rem < 1) p_rem = 1;
            if (p_rem > zk) p_rem = zk;
            const uint32_t key_p = pool_select<kLevels, true>(sh, pool, total, 0u, p_rem, a.c, M, tid);
            if (key_p > key_t) key_t = key_p;
        }
    }
    if (a.stats) {
        unsigned long long zt = 0;
        for (int i = tid; i < total; i += kThreads)
            if (pool[i] >= key_t) zt += mass_of_key(pool[i], a.c, M);
        zt = block_sum_u64(sh, zt, tid);
        if (rank == 0 && tid == 0) a.stats[row] = kept_stats(row_max, zt, finite);
    }
    key_out = key_t;
    if (kDraft) {
        // whether the row has finite mass decides, for all blocks alike, who finishes the step
        unsigned long long zt = 0;
        for (int i = tid; i < total; i += kThreads)
            if (pool[i] >= key_t) zt += mass_of_key(pool[i], a.c, M);
        zt = block_sum_u64(sh, zt, tid);
        drafted = finite && zt > 0;
        if (drafted && rank == 0) {
            __syncthreads();   // the pool is complete and the ring is idle in every warp
            draft_from_candidates(sh, pool, pool_idx, total, key_t, row_max, M, finite, a, row, scratch, tid);
        }
    }
    return true;
}

// The streaming draft step of the row at the threshold just found, for the rows the candidates
// could not finish (nucleus alone, large k, heavy ties, no finite mass).  Cluster-collective.
template <int DT>
__device__ __forceinline__ void draft_at_threshold(const ThresholdArgs& a, cg::cluster_group& cluster, int S, int rank,
                                                   int row, int tid, const RowGeom& g, uint32_t slot0, float thr) {
    DraftArgs d;
    d.logits = a.logits; d.row_stride = a.row_stride; d.V = a.V; d.c = a.c; d.thresh = a.thresh; d.greedy = 0;
    d.uniforms = a.uniforms; d.token = a.token; d.entropy = a.entropy; d.stop = a.stop;
    d.row_stats = reinterpret_cast<float*>(a.stats); d.status = a.status; d.active = nullptr;
    d.ext_target = nullptr; d.token_offset = 0; d.pos = nullptr; d.pos_stride = 0; d.slot_stride = 0; d.thr = nullptr;
    draft_row<DT, false, false, true>(d, cluster, S, rank, row, tid, g, slot0, 0, thr);
}

// kDraft: the truncated draft step in the same launch: from the candidates where that path applies,
// else by streaming the row once more at the threshold just found.
template <int DT, bool kDraft = false>
__global__ void __launch_bounds__(kThreads, 2) row_threshold_kernel(ThresholdArgs a) {
    constexpr int kLevels = DT == kBF16 ? 2 : 4;   // the low 16 bits of a bf16 logit carry nothing
    extern __shared__ uint4 ring[];
    __shared__ SelectShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int S = cluster.dim_blocks().x;
    const int rank = cluster.block_rank();
    const int row = blockIdx.x / S;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    const char* rp = static_cast<const char*>(a.logits) +
                     static_cast<size_t>(row) * a.row_stride * ElemTraits<DT>::kBytes;
    const RowGeom g = make_geom<DT>(rp, a.V, S * kWarps);
    const uint32_t slot0 = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + tid * 16;
    pdl_wait();
    if (kDraft && a.active && !a.active[row]) return;   // the whole cluster leaves together

    const bool use_k = a.top_k >= 1 && a.top_k < a.V;
    const bool use_p = a.top_p < 1.0f;
    float row_max = neg_inf();
    unsigned long long above = 0;
    bool have_max = false;
    uint32_t key_k = 0;       // key of tau_k (0: below every key, nothing dropped)

    // a small k against the number of threads of the cluster: two passes and a handful of candidates
    if (use_k && a.top_k <= (S * kThreads) / 4) {
        uint32_t key_t = 0;
        bool drafted = false, overflow = false;
        // the bound from a part of the row first (large launches); if that lets too many candidates in, from all of it
        bool done = candidate_path<DT, kDraft>(cluster, g, S, rank, tid, slot0, a, use_p, sh, key_t, ring, drafted,
                                               a.sample_den, &overflow);
        if (!done && overflow && a.sample_den > 1)
            done = candidate_path<DT, kDraft>(cluster, g, S, rank, tid, slot0, a, use_p, sh, key_t, ring, drafted, 1,
                                              &overflow);
        if (done) {
            const float thr = key_t ? key_value(key_t) : neg_inf();
            if (rank == 0 && tid == 0) a.thr[row] = thr;
            if (kDraft && !drafted) draft_at_threshold<DT>(a, cluster, S, rank, row, tid, g, slot0, thr);
            return;
        }
    }

    if (use_k) {
        uint32_t prefix = 0, k_rem = static_cast<uint32_t>(a.top_k);
        for (int level = 0; level < kLevels; ++level) {
            const int shift = 24 - 8 * level;
            if (level == 0)
                histogram_pass<DT, false, true, false>(cluster, g, S, rank, tid, slot0, prefix, shift, true, a.c, 0.f,
                                                       0u, sh, row_max, above);
            else
                histogram_pass<DT, false, false, false>(cluster, g, S, rank, tid, slot0, prefix, shift, false, a.c,
                                                        0.f, 0u, sh, row_max, above);
            if (warp == 0) decide<false>(sh, lane, k_rem, 0ull);
            __syncthreads();
            prefix |= static_cast<uint32_t>(sh.bin) << shift;
            k_rem -= sh.cnt_above;
            __syncthreads();   // the decision is read before the next pass overwrites it
        }
        have_max = true;
        // digits below the ones examined: a bf16 logit has them all zero, which the key stores as
        // ones for negative values
        key_k = prefix;
        if (DT == kBF16 && !(prefix & 0x80000000u)) key_k |= 0xffffu;
    }

    uint32_t key_t = key_k;
    if (use_p || (a.stats && !kDraft)) {
        if (!have_max) {
            // the masses are taken relative to the largest logit: find it first
            float mx = neg_inf();
            stream_segment<DT>(g, rank * kWarps + warp, lane, slot0,
                               [&](const float (&x)[ElemTraits<DT>::kEPV], int) {
#pragma unroll
                for (int j = 0; j < ElemTraits<DT>::kEPV; ++j) mx = fmaxf(mx, x[j]);
            });
            mx = warp_max(mx);
            if (lane == 0) sh.warp_max[warp] = mx;
            __syncthreads();
            if (tid == 0) {
                float m = neg_inf();
                for (int w = 0; w < kWarps; ++w) m = fmaxf(m, sh.warp_max[w]);
                sh.blk_max = m;
            }
            cluster.sync();
            float m = neg_inf();
            for (int r = 0; r < S; ++r) m = fmaxf(m, cluster.map_shared_rank(&sh, r)->blk_max);
            row_max = m;
            cluster.sync();
        }
    }
    if (use_p) {
        const bool finite = fabsf(row_max) <= kMaxLogit;
        const float M = finite ? __fmul_rn(row_max, a.c) : 0.f;
        uint32_t prefix = 0;
        unsigned long long p_rem = 0;
        for (int level = 0; level < kLevels; ++level) {
            const int shift = 24 - 8 * level;
            if (level == 0)
                histogram_pass<DT, true, false, true>(cluster, g, S, rank, tid, slot0, prefix, shift, true, a.c, M,
                                                      key_k, sh, row_max, above);
            else
                histogram_pass<DT, true, false, false>(cluster, g, S, rank, tid, slot0, prefix, shift, false, a.c, M,
                                                       key_k, sh, row_max, above);
            if (level == 0) {
                // target mass: top_p of the mass of the top-k set (the whole row without top-k)
                const double want = ceil(static_cast<double>(a.top_p) * static_cast<double>(above));
                p_rem = static_cast<unsigned long long>(want);
                if (p_rem < 1) p_rem = 1;
                if (p_rem > above) p_rem = above;
            }
            if (warp == 0) decide<true>(sh, lane, 0u, p_rem);
            __syncthreads();
            prefix |= static_cast<uint32_t>(sh.bin) << shift;
            p_rem -= sh.mass_above;
            __syncthreads();
        }
        uint32_t key_p = prefix;
        if (DT == kBF16 && !(prefix & 0x80000000u)) key_p |= 0xffffu;
        if (above == 0 || !finite) key_p = 0;   // a row without mass: the nucleus drops nothing
        key_t = key_p > key_k ? key_p : key_k;
    }
    if (rank == 0 && tid == 0) a.thr[row] = key_t ? key_value(key_t) : neg_inf();
    if (kDraft) {
        draft_at_threshold<DT>(a, cluster, S, rank, row, tid, g, slot0, key_t ? key_value(key_t) : neg_inf());
        return;
    }
    if (a.stats && !kDraft) {
        // the mass of the kept set: one more pass (the descents above know it only in part)
        const bool finite = fabsf(row_max) <= kMaxLogit;
        const float M = finite ? __fmul_rn(row_max, a.c) : 0.f;
        unsigned long long kept = 0;
        stream_segment<DT>(g, rank * kWarps + warp, lane, slot0, [&](const float (&x)[ElemTraits<DT>::kEPV], int) {
#pragma unroll
            for (int j = 0; j < ElemTraits<DT>::kEPV; ++j) {
                if (order_key(x[j]) >= key_t) {
                    const float w = ex2_approx(fmaxf(__fmaf_rn(x[j], a.c, -M), kArgFloor));
                    kept += __float2ull_rz(w * kMassScale);
                }
            }
        });
        kept = block_sum_u64(sh, kept, tid);
        if (tid == 0) sh.blk_above = kept;
        cluster.sync();
        unsigned long long all = 0;
        for (int r = 0; r < S; ++r) all += cluster.map_shared_rank(&sh, r)->blk_above;
        if (rank == 0 && tid == 0) a.stats[row] = kept_stats(row_max, all, finite);
        cluster.sync();   // the peers have read this block's sum
    }
    // every pass ended with a cluster barrier after all remote reads: blocks may leave
}

}  // namespace svip
