// Small kernels around the hot path: vocabulary-parallel combine, draft-length policies, ragged packing.
#pragma once

#include "svip_draft.cuh"

namespace svip {
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

// One block waits on an mbarrier that expects bytes nobody sends, with the bounded wait of the
// cluster exchange, and reports the time-out in the status word (svip_selftest_wait_timeout).
__global__ void __launch_bounds__(32) wait_timeout_kernel(unsigned long long wait_ns, unsigned* status) {
    __shared__ unsigned long long bar;
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t b = static_cast<uint32_t>(__cvta_generic_to_shared(&bar));
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        mbar_arrive_expect_tx(b, 16);
    }
    __syncwarp();
    if (!mbar_wait_bounded(b, 0, wait_ns) && threadIdx.x == 0) atomicOr(status, SVIP_STATUS_WAIT_TIMEOUT);
}

}  // namespace svip
