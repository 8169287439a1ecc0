// Device-side building blocks shared by the SVIP kernels (sm_100a).
//
// A logits row is streamed once from HBM with 128-bit loads.  The row is cut
// into NSEG = (blocks per cluster) x (warps per block) contiguous segments, one
// per warp, so that a warp's partial sum is the mass of a contiguous index
// range: inverse-CDF sampling then only has to re-read ONE segment (an L2 hit)
// after the normaliser is known, instead of the whole row.
//
// Per-thread state while streaming (fast path):
//   rmax running maximum of the raw logits (exact in fp32), tracked without branches
//   ref  reference logit of the exponentials; Mref = rn(ref*c), c = log2(e)/T
//   Z    sum of 2^(x*c - Mref)                      (two packed fp32 accumulators)
//   A    sum of 2^(x*c - Mref) * (x*c - Mref)       (log2 units, for the entropy)
// The reference is NOT kept equal to the running maximum: it starts as the largest logit among the
// warp's first vectors and is only moved up (and Z, A rescaled) when the maximum has run more than
// 2^64 ahead of it, checked once per kStages vectors, which almost never happens, so the warp does
// not diverge on the common "some lane saw a new maximum" event.  Exponents up to +64 are harmless
// in fp32; a larger jump between two checks overflows to inf and sends the warp to the slow path.
// Partials merge by rescaling to the larger maximum.
//
// Loads go through a per-thread ring of cp.async slots in shared memory (kStages x 16 bytes per
// thread): up to kStages loads per thread stay in flight while the thread computes, with no
// registers held and no barriers (a thread only reads the slots it filled itself).
//
// The fast path has no special cases: -inf logits make 0 * -inf = NaN in A and NaN logits make
// NaN in Z, and a warp whose result is NaN redoes its segment on the slow path, which masks
// such logits to zero mass.
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace svip {

namespace cg = cooperative_groups;

constexpr int kWarps = 16;              // warps per thread block
constexpr int kThreads = kWarps * 32;   // threads per thread block
constexpr int kMaxCluster = 8;          // portable cluster size limit
constexpr int kMaxSeg = kMaxCluster * kWarps;
constexpr int kSegPerLane = kMaxSeg / 32;
constexpr int kF32 = 0;
constexpr int kBF16 = 1;
constexpr float kArgFloor = -127.0f;    // 2^x flushes to zero below this (ftz)
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kIntMax = 0x7fffffff;
constexpr int kStages = 8;              // cp.async slots per thread
constexpr int kRingBytes = kStages * kThreads * 16;
constexpr float kRebase = 64.0f;        // move the reference when the maximum is 2^64 ahead of it
constexpr float kMasked = -1.0e30f;     // fast-path stand-in for elements outside the row
constexpr float kMaxLogit = 1.0e29f;    // rows whose maximum lies outside +-1e29 are reported as non-finite

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// Bounds-checked build (-DSVIP_DEBUG_BOUNDS): every global load of logits (the ring's cp.async copies, the
// streaming vector loads, the single-element gathers) is checked against the extents of the logits buffers
// of the call, which the host puts into constant memory before the launch.  A load outside is not
// performed (zeros are used) and counted; svip_read_status then reports SVIP_STATUS_DEBUG_OOB.  Stands in
// for a memory checker where none can be run.
#ifdef SVIP_DEBUG_BOUNDS
struct DebugRange { unsigned long long lo, hi; };
__constant__ DebugRange g_debug_range[2];
__device__ unsigned g_debug_oob;
__device__ __forceinline__ bool debug_ok(const void* p, unsigned bytes) {
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
    const bool ok = (a >= g_debug_range[0].lo && a + bytes <= g_debug_range[0].hi) ||
                    (a >= g_debug_range[1].lo && a + bytes <= g_debug_range[1].hi);
    if (!ok) atomicAdd(&g_debug_oob, 1u);
    return ok;
}
#else
__device__ __forceinline__ bool debug_ok(const void*, unsigned) { return true; }
#endif

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 128-bit streaming load: read-only path, no L1 allocation (each byte is used once).
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    if (!debug_ok(p, 16)) return make_uint4(0, 0, 0, 0);
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 128-bit load through the read-only path that may be reused (second touches: fine scans, residual rows).
__device__ __forceinline__ uint4 ld_vec(const uint4* p) {
    if (!debug_ok(p, 16)) return make_uint4(0, 0, 0, 0);
    return __ldg(p);
}

template <int DT> struct ElemTraits;
template <> struct ElemTraits<kF32> {
    static constexpr int kEPV = 4;      // elements per 16-byte vector
    static constexpr int kBytes = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float load_one(const void* row, int i) {
        if (!debug_ok(reinterpret_cast<const float*>(row) + i, 4)) return 0.f;
        return __ldg(reinterpret_cast<const float*>(row) + i);
    }
};
template <> struct ElemTraits<kBF16> {
    static constexpr int kEPV = 8;
    static constexpr int kBytes = 2;
    // bfloat16 is the upper half of an fp32: element 2k sits in the low half-word.
    __device__ static __forceinline__ void unpack(const uint4& v, float (&x)[8]) {
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
    __device__ static __forceinline__ float load_one(const void* row, int i) {
        if (!debug_ok(reinterpret_cast<const unsigned short*>(row) + i, 2)) return 0.f;
        unsigned short h = __ldg(reinterpret_cast<const unsigned short*>(row) + i);
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
};

// Geometry of one row seen as 16-byte vectors.  The row may start anywhere:
// the vectors start at the 16-byte boundary at or below the first element, and
// `pre` counts the elements of the first vector that lie before the row.
// Those, and the elements of the last vector past the row, are masked to -inf.
// (They lie in the same 16-byte granule as valid data, so the load is safe.)
struct RowGeom {
    const uint4* base;
    int pre;    // leading pad elements in vector 0
    int V;      // valid elements
    int nvec;   // vectors covering [0, pre + V)
    int vps;    // vectors per segment (multiple of 8 = one 128-byte line)
};

template <int DT>
__device__ __forceinline__ RowGeom make_geom(const void* row, int V, int nseg) {
    using E = ElemTraits<DT>;
    RowGeom g;
    uintptr_t p = reinterpret_cast<uintptr_t>(row);
    int mis = static_cast<int>(p & 15);
    g.base = reinterpret_cast<const uint4*>(p - mis);
    g.pre = mis / E::kBytes;
    g.V = V;
    g.nvec = (g.pre + V + E::kEPV - 1) / E::kEPV;
    int vps = (g.nvec + nseg - 1) / nseg;
    g.vps = (vps + 7) & ~7;
    return g;
}

__device__ __forceinline__ void seg_range(const RowGeom& g, int seg, int& v_lo, int& v_hi) {
    long lo = static_cast<long>(seg) * g.vps;
    v_lo = lo < g.nvec ? static_cast<int>(lo) : g.nvec;
    v_hi = min(v_lo + g.vps, g.nvec);
}

// Unpacks vector vi of the row and masks the elements outside the row to -inf.
template <int DT>
__device__ __forceinline__ void unpack_masked(const uint4& raw, int vi, const RowGeom& g,
                                              float (&x)[ElemTraits<DT>::kEPV]) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    ElemTraits<DT>::unpack(raw, x);
    if (vi == 0 || vi == g.nvec - 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            int e = vi * EPV + j;
            if (e < g.pre || e >= g.pre + g.V) x[j] = neg_inf();
        }
    }
}

struct Partial {
    float m;   // maximum raw logit (-inf if nothing seen)
    int idx;   // lowest index attaining m (kIntMax if nothing seen)
    float Z;   // mass relative to rn(m*c)
    float A;   // sum of mass * log2-argument, relative to rn(m*c)
};

template <int EPV>
__device__ __forceinline__ float vec_max(const float (&x)[EPV]) {
    float t = fmaxf(x[0], x[1]);
#pragma unroll
    for (int j = 2; j < EPV; ++j) t = fmaxf(t, x[j]);
    return t;
}

// Folds one vector into the thread's partial.  kMode: 0 = max/argmax only,
// 1 = max + Z, 2 = max + Z + A.
template <int DT, int kMode>
__device__ __forceinline__ void fold_vector(const uint4& raw, int vi, const RowGeom& g, float c,
                                            Partial& t, float& M, float thr = -INFINITY) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    float x[EPV];
    unpack_masked<DT>(raw, vi, g, x);
#pragma unroll
    for (int j = 0; j < EPV; ++j)
        if (!(x[j] >= thr)) x[j] = neg_inf();   // below the truncation threshold (or NaN): dropped
    float tmax = vec_max<EPV>(x);
    if (tmax > t.m) {
        float Mn = __fmul_rn(tmax, c);
        if (kMode >= 1 && t.m != neg_inf()) {
            float d = M - Mn;
            float s = ex2_approx(fmaxf(d, kArgFloor));
            if (kMode == 2) t.A = s * __fmaf_rn(d, t.Z, t.A);
            t.Z *= s;
        }
        int first = 0;
#pragma unroll
        for (int j = EPV - 1; j >= 0; --j)
            if (x[j] == tmax) first = j;
        t.m = tmax;
        t.idx = vi * EPV + first - g.pre;
        M = Mn;
    }
    if (kMode >= 1) {
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            float a = fmaxf(__fmaf_rn(x[j], c, -M), kArgFloor);   // NaN -> floor: zero mass
            float e = ex2_approx(a);
            t.Z += e;
            if (kMode == 2) t.A = __fmaf_rn(e, a, t.A);
        }
    }
}

// Slow path: streams segment `seg` with plain loads, an exact per-lane running maximum and
// masking of -inf / NaN logits to zero mass.
template <int DT, int kMode>
__device__ __noinline__ Partial reduce_segment_slow(const RowGeom& g, int seg, float c, int lane,
                                                    float thr = -INFINITY) {
    Partial t;
    t.m = neg_inf(); t.idx = kIntMax; t.Z = 0.f; t.A = 0.f;
    float M = neg_inf();
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    for (int vi = v_lo + lane; vi < v_hi; vi += 32) {
        uint4 r0 = ld_stream(g.base + vi);
        fold_vector<DT, kMode>(r0, vi, g, c, t, M, thr);
    }
    return t;
}

// ---------------------------------------------------------------------------
// Fast path: cp.async ring + packed fp32x2 arithmetic.

__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* gptr) {
    if (!debug_ok(gptr, 16)) return;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(gptr) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(saddr)
                 : "memory");
    return v;
}

// Programmatic dependent launch: a kernel lets the next kernel of the stream be scheduled at once
// (its blocks become resident and run their prologue) and itself waits, before it touches global
// memory, until the previous kernel has completed and flushed.  Both are no-ops for a kernel that
// was launched without the programmatic-serialization attribute.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Split cluster barrier: arrive as soon as this thread is done with its peers' shared memory,
// wait only before leaving (a block must not exit while a peer may still read its memory).
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Exchange of segment partials inside a cluster without a closing barrier: every warp pushes its
// 16-byte entry into the shared memory of every block of the cluster (st.async through distributed
// shared memory), and each push counts its bytes on the receiving block's mbarrier.  A block then
// only waits on its own mbarrier until all entries of the cluster have landed: one one-way trip
// instead of a barrier round trip followed by remote reads.  Nothing is read remotely, so a block may
// leave as soon as its own mbarrier has completed (all writes aimed at it have arrived by then).

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n"
        " mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        " selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // one second: far beyond any exchange, short for a hang

// Waits for the phase `parity` of the mbarrier, at most limit_ns nanoseconds.  Returns false if the
// time ran out (the caller records it in the status word and carries on with what it has).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}
// Address of the same shared-memory location in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
// 16 bytes into a peer's shared memory; the peer's mbarrier is credited with 16 bytes when they land.
__device__ __forceinline__ void push16(uint32_t remote_addr, uint32_t remote_bar, uint32_t a, uint32_t b,
                                       uint32_t c, uint32_t d) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(remote_bar) : "memory");
}

typedef unsigned long long f32x2;   // two packed fp32 values
__device__ __forceinline__ f32x2 pack2(float a, float b) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

struct Acc {
    float rmax;    // running maximum of the raw logits
    int ivec;      // vector that first attained rmax (tracked only when asked for)
    float Mref;    // rn(reference logit * c)
    f32x2 c2;      // (c, c)
    f32x2 nm2;     // (-Mref, -Mref)
    f32x2 Z2;
    f32x2 A2;
};

__device__ __forceinline__ void acc_init(Acc& t, float ref, float c) {
    t.rmax = neg_inf(); t.ivec = kIntMax; t.Mref = __fmul_rn(ref, c);
    t.c2 = pack2(c, c); t.nm2 = pack2(-t.Mref, -t.Mref);
    t.Z2 = pack2(0.f, 0.f); t.A2 = pack2(0.f, 0.f);
}

// Moves the reference up to the running maximum.
template <int kMode>
__device__ __forceinline__ void acc_rebase(Acc& t, float c) {
    float Mn = __fmul_rn(t.rmax, c);
    float d = t.Mref - Mn;
    float s = ex2_approx(fmaxf(d, kArgFloor));
    f32x2 s2 = pack2(s, s);
    if (kMode == 2) t.A2 = mul2(s2, fma2(pack2(d, d), t.Z2, t.A2));
    t.Z2 = mul2(s2, t.Z2);
    t.Mref = Mn;
    t.nm2 = pack2(-Mn, -Mn);
}

// Folds EPV unpacked logits (no special values expected) into the accumulator.  The reference is
// not touched here; the caller checks now and then whether it has to move (acc_check).
template <int EPV, int kMode, bool kIdx>
__device__ __forceinline__ void fold_fast(const float (&x)[EPV], int vi, Acc& t) {
    float old = t.rmax;
    if (EPV == 8) {
        float a = max3(old, x[0], x[1]);
        float b = max3(x[2], x[3], x[4]);
        float d = max3(x[5], x[6], x[7]);
        t.rmax = max3(a, b, d);
    } else {
        float a = max3(old, x[0], x[1]);
        t.rmax = max3(a, x[2], x[3]);
    }
    if (kIdx) {
        if (t.rmax > old) t.ivec = vi;
    }
    if (kMode >= 1) {
#pragma unroll
        for (int j = 0; j < EPV; j += 2) {
            f32x2 a2 = fma2(pack2(x[j], x[j + 1]), t.c2, t.nm2);
            float a0, a1;
            unpack2(a2, a0, a1);
            f32x2 e2 = pack2(ex2_approx(a0), ex2_approx(a1));
            t.Z2 = add2(t.Z2, e2);
            if (kMode == 2) t.A2 = fma2(e2, a2, t.A2);
        }
    }
}

// Moves the reference up if the running maximum has run far ahead of it.
template <int kMode>
__device__ __forceinline__ void acc_check(Acc& t, float c) {
    if (kMode == 0) return;
    if (__fmaf_rn(t.rmax, c, -t.Mref) > kRebase) acc_rebase<kMode>(t, c);
}

// Unpacks vector vi and replaces the elements outside the row by a very negative finite value.
template <int DT>
__device__ __forceinline__ void unpack_edge(const uint4& raw, int vi, const RowGeom& g,
                                            float (&x)[ElemTraits<DT>::kEPV]) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    ElemTraits<DT>::unpack(raw, x);
#pragma unroll
    for (int j = 0; j < EPV; ++j) {
        int e = vi * EPV + j;
        if (e < g.pre || e >= g.pre + g.V) x[j] = kMasked;
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ int warp_min_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Rescales a partial from its own maximum to the maximum m_to (m_to >= t.m).
template <int kMode>
__device__ __forceinline__ void rescale_to(Partial& t, float m_to, float c) {
    if (kMode == 0) return;
    if (t.m == neg_inf() || !(t.Z > 0.f)) { t.Z = 0.f; t.A = 0.f; return; }
    float d = __fmul_rn(t.m, c) - __fmul_rn(m_to, c);
    float s = ex2_approx(fmaxf(d, kArgFloor));
    if (kMode == 2) t.A = s * __fmaf_rn(d, t.Z, t.A);
    t.Z *= s;
}

// All lanes return the merge of the 32 lanes' partials.
template <int kMode>
__device__ __forceinline__ Partial warp_merge(Partial t, float c) {
    float m = warp_max(t.m);
    int idx = warp_min_int(t.m == m ? t.idx : kIntMax);
    rescale_to<kMode>(t, m, c);
    Partial r;
    r.m = m; r.idx = idx;
    r.Z = kMode >= 1 ? warp_sum(t.Z) : 0.f;
    r.A = kMode == 2 ? warp_sum(t.A) : 0.f;
    return r;
}

// Streams segment `seg` of the row with the calling warp and returns the warp's merged partial
// (all lanes hold it).  `slot0` is the shared-memory address of this thread's first ring slot;
// slot s lives kThreads * 16 bytes further.  kIdx asks for the index of the maximum.
// Logits below the truncation threshold get the stand-in that carries no mass.
template <int EPV>
__device__ __forceinline__ void drop_below(float (&x)[EPV], float thr) {
#pragma unroll
    for (int j = 0; j < EPV; ++j) x[j] = x[j] >= thr ? x[j] : kMasked;
}

// kThr: only logits >= thr count (truncated distributions); the reference of the exponentials is
// still taken from the raw logits, so a segment without a kept logit simply sums to zero.
template <int DT, int kMode, bool kIdx, bool kThr = false>
__device__ __forceinline__ Partial reduce_segment(const RowGeom& g, int seg, float c, int lane,
                                                  uint32_t slot0, float thr = -INFINITY) {
    constexpr int EPV = ElemTraits<DT>::kEPV;
    constexpr uint32_t kSlotStride = kThreads * 16;
    int v_lo, v_hi;
    seg_range(g, seg, v_lo, v_hi);
    // vectors that stick out of the row are folded apart, by lane 0, with their outside masked
    const bool head_edge = g.pre > 0;
    const bool tail_edge = ((g.pre + g.V) % EPV) != 0;
    int i_lo = v_lo, i_hi = v_hi;
    if (head_edge && v_lo == 0 && v_hi > 0) i_lo = 1;
    if (tail_edge && v_hi == g.nvec && i_hi > i_lo) i_hi = g.nvec - 1;
    const bool fold_head = lane == 0 && head_edge && v_lo == 0 && v_hi > 0;
    const bool fold_tail = lane == 0 && tail_edge && v_hi == g.nvec && v_lo < v_hi && !(g.nvec == 1 && head_edge);
    const int vi0 = i_lo + lane;
    const int n = i_hi > vi0 ? (i_hi - vi0 + 31) >> 5 : 0;
    const uint4* src = g.base + vi0;
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
        if (s < n) cp_async16(slot0 + s * kSlotStride, src + 32 * s);
        cp_async_commit();
    }
    // The reference of the exponentials: the largest logit among the warp's first vectors, the
    // same for all lanes.  Later logits may exceed it by up to 2^kRebase before it is moved.
    float ref = 0.f;
    bool bad = false;
    if (kMode >= 1) {
        float fm = neg_inf();
        if (fold_head) {
            float x[EPV];
            unpack_masked<DT>(ld_stream(g.base), 0, g, x);
            fm = vec_max<EPV>(x);
        }
        if (fold_tail) {
            float x[EPV];
            unpack_masked<DT>(ld_stream(g.base + g.nvec - 1), g.nvec - 1, g, x);
            fm = fmaxf(fm, vec_max<EPV>(x));
        }
        cp_async_wait<kStages - 1>();
        if (n > 0) {
            float x[EPV];
            ElemTraits<DT>::unpack(lds128(slot0), x);
            fm = fmaxf(fm, vec_max<EPV>(x));
        }
        ref = warp_max(fm);
        bad = !(fabsf(ref) <= kMaxLogit);   // nothing finite seen (or +inf): leave it to the slow path
    }
    Acc t;
    acc_init(t, ref, c);
    if (!bad) {
        if (fold_head) {
            float x[EPV];
            unpack_edge<DT>(ld_stream(g.base), 0, g, x);
            if (kThr) drop_below<EPV>(x, thr);
            fold_fast<EPV, kMode, kIdx>(x, 0, t);
        }
        int it = 0;
        // steady state: every prefetch is in range, slot numbers are compile-time constants
        for (; it + 2 * kStages <= n; it += kStages) {
            const uint4* p = src + 32 * it;
#pragma unroll
            for (int s = 0; s < kStages; ++s) {
                cp_async_wait<kStages - 1>();
                const uint4 raw = lds128(slot0 + s * kSlotStride);
                cp_async16(slot0 + s * kSlotStride, p + 32 * (kStages + s));
                cp_async_commit();
                float x[EPV];
                ElemTraits<DT>::unpack(raw, x);
                if (kThr) drop_below<EPV>(x, thr);
                fold_fast<EPV, kMode, kIdx>(x, vi0 + 32 * (it + s), t);
            }
            acc_check<kMode>(t, c);
        }
        // last full ring: same static slots, prefetches only where the segment still has vectors
        for (; it + kStages <= n; it += kStages) {
            const uint4* p = src + 32 * it;
#pragma unroll
            for (int s = 0; s < kStages; ++s) {
                cp_async_wait<kStages - 1>();
                const uint4 raw = lds128(slot0 + s * kSlotStride);
                if (it + kStages + s < n) cp_async16(slot0 + s * kSlotStride, p + 32 * (kStages + s));
                cp_async_commit();
                float x[EPV];
                ElemTraits<DT>::unpack(raw, x);
                if (kThr) drop_below<EPV>(x, thr);
                fold_fast<EPV, kMode, kIdx>(x, vi0 + 32 * (it + s), t);
            }
            acc_check<kMode>(t, c);
        }
        // fewer than kStages vectors left, all of them already in flight: `it` is a multiple of
        // kStages, so vector it + k sits in slot k
        cp_async_wait<0>();
        for (; it < n; ++it) {
            const uint4 raw = lds128(slot0 + (it & (kStages - 1)) * kSlotStride);
            float x[EPV];
            ElemTraits<DT>::unpack(raw, x);
            if (kThr) drop_below<EPV>(x, thr);
            fold_fast<EPV, kMode, kIdx>(x, vi0 + 32 * it, t);
        }
        acc_check<kMode>(t, c);
        if (fold_tail) {
            float x[EPV];
            unpack_edge<DT>(ld_stream(g.base + g.nvec - 1), g.nvec - 1, g, x);
            if (kThr) drop_below<EPV>(x, thr);
            fold_fast<EPV, kMode, kIdx>(x, g.nvec - 1, t);
            acc_check<kMode>(t, c);
        }
    }
    cp_async_wait<0>();

    float z0, z1, a0, a1;
    unpack2(t.Z2, z0, z1);
    unpack2(t.A2, a0, a1);
    float Z = z0 + z1, A = a0 + a1;
    // +inf, NaN (from -inf or NaN logits, or an overflow between two checks): redo the segment
    if (kMode >= 1) bad = bad || !(fabsf(Z) <= 3.0e38f) || !(fabsf(A) <= 3.0e38f);
    if (__any_sync(0xffffffffu, bad)) {
        Partial p = reduce_segment_slow<DT, kMode>(g, seg, c, lane, kThr ? thr : -INFINITY);
        return warp_merge<kMode>(p, c);
    }
    Partial r;
    r.m = warp_max(t.rmax);
    r.idx = kIntMax;
    r.Z = 0.f; r.A = 0.f;
    if (kMode >= 1) {
        if (Z > 0.f) {
            float d = t.Mref - __fmul_rn(r.m, c);
            float sc = ex2_approx(fmaxf(d, kArgFloor));
            if (kMode == 2) A = sc * __fmaf_rn(d, Z, A);
            Z *= sc;
        } else {
            Z = 0.f; A = 0.f;
        }
        r.Z = warp_sum(Z);
        if (kMode == 2) r.A = warp_sum(A);
    }
    if (kIdx) {
        int iv = warp_min_int(t.rmax == r.m ? t.ivec : kIntMax);
        if (iv != kIntMax) {
            float x[EPV];
            unpack_masked<DT>(ld_vec(g.base + iv), iv, g, x);
            int first = -1;
#pragma unroll
            for (int j = EPV - 1; j >= 0; --j)
                if (x[j] == r.m) first = j;
            if (first >= 0) r.idx = iv * EPV + first - g.pre;
        }
    }
    return r;
}

// Inclusive warp scan.
__device__ __forceinline__ float warp_scan_incl(float v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        float n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

// Block-wide exclusive scan of one float per thread; also returns the block total.
// `wsum` is shared scratch of kWarps floats.  Contains two __syncthreads().
__device__ __forceinline__ float block_scan_excl(float v, float* wsum, int lane, int warp, float& total) {
    float inc = warp_scan_incl(v, lane);
    __syncthreads();   // wsum may still be read from the previous round
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    float before = 0.f, tot = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        float s = wsum[w];
        if (w < warp) before += s;
        tot += s;
    }
    total = tot;
    return before + (inc - v);
}

// ---------------------------------------------------------------------------
// Locating a sample among the segments of a row.
//
// Each block of the cluster publishes, per warp, the mass of its segment in
// shared memory.  Warp 0 of EVERY block then reads all segments of the cluster
// through distributed shared memory, in the same order with the same
// arithmetic, so all blocks agree bit for bit on the total, on the target mass
// u * total and on the segment that holds it; the block that owns the segment
// does the fine scan.

struct SegPick {
    float total;    // sum of all segment masses = last inclusive prefix
    int seg;        // selected segment
    float prefix;   // exclusive prefix of the selected segment
    float target;   // u * total
};

// `mass[k]` is the mass of segment lane*per + k (0 beyond nseg).  Warp-collective.
// The mass to find is u * total, or `abs_target` (same units as the masses) when that is >= 0.
__device__ __forceinline__ SegPick pick_segment(const float (&mass)[kSegPerLane], int per, int nseg,
                                                float u, int lane, float abs_target = -1.f) {
    float run[kSegPerLane];
    float acc = 0.f;
#pragma unroll
    for (int k = 0; k < kSegPerLane; ++k) {
        if (k < per) acc += mass[k];
        run[k] = acc;                       // inclusive within the lane
    }
    float incl = warp_scan_incl(acc, lane);
    float before = incl - acc;
    SegPick r;
    r.total = __shfl_sync(0xffffffffu, incl, 31);
    r.target = abs_target >= 0.f ? abs_target : u * r.total;
    int cand = kIntMax;
    float cpre = 0.f;
#pragma unroll
    for (int k = kSegPerLane - 1; k >= 0; --k) {
        if (k < per && lane * per + k < nseg && before + run[k] > r.target) {
            cand = lane * per + k;
            cpre = before + (run[k] - mass[k]);
        }
    }
    int best = warp_min_int(cand);
    if (best == kIntMax) {
        // rounding left no prefix above the target: take the last segment with mass
        int lastpos = -1;
        float lpre = 0.f;
#pragma unroll
        for (int k = 0; k < kSegPerLane; ++k) {
            if (k < per && lane * per + k < nseg && mass[k] > 0.f) {
                lastpos = lane * per + k;
                lpre = before + (run[k] - mass[k]);
            }
        }
        int hi = -warp_min_int(-lastpos);
        best = hi < 0 ? 0 : hi;
        cand = (lastpos == best) ? best : kIntMax;
        cpre = lpre;
    }
    unsigned who = __ballot_sync(0xffffffffu, cand == best);
    int src = who ? __ffs(who) - 1 : 0;
    r.seg = best;
    r.prefix = __shfl_sync(0xffffffffu, cpre, src);
    return r;
}

// Shared scratch of the fine scan.
struct ScanShared {
    float wsum[kWarps];
    unsigned long long key;   // (lowest thread whose run crosses the target) << 32 | the element it found
    int lastpos;              // highest vector with positive weight
    int result;               // the element found on the fallback path
};

}  // namespace svip
