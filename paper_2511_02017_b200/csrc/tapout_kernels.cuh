// Kernels of libtapout (sm_100a).  The two streaming kernels read each needed logit row from HBM
// exactly once with 128-bit coalesced loads; everything per-row that is scalar runs in double.
//
//   k_draft_step    one launch per draft position: a persistent grid strides over (row, segment)
//                   items; the CTA that reduces the last segment of a row also finishes the row
//                   (features, token draw, stop rule, bookkeeping), so no second launch is needed.
//   k_verify_walk   one thread-block cluster per sequence: every CTA streams its slice of the target
//                   row, the per-warp partial sums are exchanged through distributed shared memory,
//                   and all CTAs take the same accept / reject decision before the next row.
//   k_update        rewards, arm statistics, AdaEDL, and the arm choices of the next round.
#pragma once

#include <cooperative_groups.h>

#include "tapout_device.cuh"

namespace tpo {

namespace cg = cooperative_groups;

constexpr int kMaxCluster = 8;           // portable cluster size limit
constexpr int kResident = 4;              // CTAs of a streaming kernel resident per SM (64 registers per thread)
constexpr int kTodo = 32;                // rows a CTA may queue for finishing after its streaming loop

struct WarpRec { float ref, k, S, T, c1, c2; int best; int pad; };

// How many CTAs share one draft row, decided on the device from the number of rows actually drafted at
// this position (the host never learns it): the smallest split whose items fill at least 90 % of a whole
// number of waves of the persistent grid, else the best-filling one; never less than a chunk per warp.
__device__ __forceinline__ int segments_for(const Params& p, int n_rows, int grid) {
    if (p.nseg > 0) return p.nseg;
    const unsigned cap = (unsigned)max(1, min(min(kMaxSeg, p.NC), max(p.NC / kWarps, 1)));
    if (n_rows <= 0) return 1;
    const unsigned n = (unsigned)n_rows, G = (unsigned)grid;     // n * cap < 2^31: n_seq is bounded at create
    unsigned best = 1;
    float best_fill = 0.f;
    for (unsigned k = 1; k <= cap; ++k) {
        const unsigned items = n * k;
        const unsigned slots = (items + G - 1) / G * G;
        const float fill = (float)items / (float)slots;
        if (fill >= 0.9f) return (int)k;
        if (fill > best_fill) { best = k; best_fill = fill; }
    }
    return (int)best;
}

// One warp's share of the chunks [c0, c1) of a row: chunk c0 + warp, then every kWarps-th.  Loads are not
// staged ahead: with four CTAs resident per SM the other warps cover the latency, and the registers a
// second buffer would take cost more than it gains.  store(ch, ref, total) receives the per-chunk partial
// sum when WANT_PART.
template <int DT, bool WANT_T, bool WANT_PART, typename Store>
__device__ __forceinline__ void stream_chunks(WarpAcc& acc, const void* row, int V, int c0, int c1, int warp, int lane,
                                              float c, Store store) {
    for (int ch = c0 + warp; ch < c1; ch += kWarps) {
        uint4 v[kVecPerLane];
        load_chunk<DT>(row, V, ch, lane, v);
        const float tot = fold_chunk<DT, WANT_T, WANT_PART>(acc, v, ch, c);
        if (WANT_PART && lane == 0) store(ch, acc.ref, tot);
    }
}

// What the finishing warp needs besides Params / State / Scratch.
struct StepArgs {
    const void* logits;
    long long row_stride;
    int pos, slot, n_fixed, grid_ref;
    uint32_t round;
    float c, inv_T;
    int32_t* out_token;
    long long tok_stride;
    uint8_t* out_continue;
    float* out_feat;
};

__device__ __forceinline__ SegRec load_segrec(const SegRec* g) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(g));
    const int4 b = __ldcg(reinterpret_cast<const int4*>(g) + 1);
    SegRec r;
    r.ref = a.x; r.S = a.y; r.T = a.z; r.c2 = a.w; r.best = b.x; r.pad0 = r.pad1 = r.pad2 = 0;
    return r;
}

__device__ __forceinline__ void store_segrec(SegRec* g, const SegRec& r) {
    reinterpret_cast<float4*>(g)[0] = make_float4(r.ref, r.S, r.T, r.c2);
    reinterpret_cast<int4*>(g)[1] = make_int4(r.best, 0, 0, 0);
}

// Finishes one row once all of its segments are reduced (one warp).  Draft position: Table 1 features,
// x_i ~ softmax(row), the stop rule of the arm chosen for this position, bookkeeping, and the list for
// the next position.  FEATURES (tapout_row_stats): the features only, nothing of the round's state is
// touched.  Two dependent trips to memory: the segment records with the chunk partials, then the two
// 2 KB chunks that hold the row maximum and the drawn token.
template <int DT, bool FEATURES>
__device__ __forceinline__ void finish_row(const Params& p, const State& st, const Scratch& sc, const StepArgs& a, int s,
                                        int nseg, int lane) {
    const char* row = reinterpret_cast<const char*>(a.logits) + (size_t)s * a.row_stride * Elem<DT>::BYTES;
    const float2* part = sc.cdf + (size_t)s * p.NC;
    const float c = a.c;
    const int pos = a.pos;

    // ---- segment records and chunk partials
    SegRec r;
    r.ref = neg_inf(); r.S = 0.f; r.T = 0.f; r.c2 = neg_inf(); r.best = -1;
    if (lane < nseg) r = load_segrec(sc.seg + (size_t)s * kMaxSeg + lane);
    const bool in_regs = p.NC <= 32 * kRegPer;
    RegCdf cdf;
    if (in_regs) cdf.load(part, p.NC, lane);
    const bool has_nan = __any_sync(0xffffffffu, (r.S != r.S) || (r.T != r.T) || (r.ref != r.ref));
    const float m = warp_max_f(r.ref);
    const double mc = (double)m * (double)c;
    double Tg = 0.0;
    if (lane < nseg && r.ref > neg_inf() && r.ref < CUDART_INF_F) {
        const double d = (double)__fmul_rn(-r.ref, c) + mc;              // >= 0 up to rounding
        Tg = exp2(-d) * ((double)r.T - d * (double)r.S);
    }
    const double T2 = warp_sum_d(Tg);                                    // sum of w * t (log2 units)
    CdfTotals tot;
    double W;
    if (in_regs) { cdf.scale(c, mc, lane); W = cdf.W; }
    else { tot = cdf_totals<true>(part, p.NC, c, mc, true, lane); W = tot.W; }
    const bool valid = !has_nan && (m > neg_inf()) && (m < CUDART_INF_F) && (W > 0.0) && (W < CUDART_INF);

    if (lane == 0) sc.done[s] = 0;
    if (!FEATURES && lane == 0) atomicAdd(&sc.status[1], 1ull);
    if (!valid) {
        if (lane == 0) {
            if (FEATURES) {
                float* fo = a.out_feat + (size_t)s * kFeat;
                const float qn = __int_as_float(0x7fc00000);
                fo[0] = fo[1] = fo[2] = fo[3] = fo[4] = qn; fo[5] = -1.f;
            } else {
                atomicOr(&sc.status[0], 1ull);
                a.out_token[(size_t)s * a.tok_stride] = -1; a.out_continue[s] = 0; st.active[s] = 0;
                sc.stopped[atomicAdd(&sc.count[3], 1)] = s;
            }
        }
        return;
    }

    // ---- which chunk holds the maximum (lowest such), which one the drawn token
    const unsigned tie = __ballot_sync(0xffffffffu, lane < nseg && r.ref == m);
    const int win = __ffs(tie) - 1;
    const float other = warp_max_f((lane == win || lane >= nseg) ? neg_inf() : r.ref);
    const float c2all = warp_max_f(r.c2);
    const int best = max(__shfl_sync(0xffffffffu, r.best, win), 0);
    int chunk = 0;
    double rem = 0.0;
    float refc = 0.f;
    if (!FEATURES) {
        const uint32_t seq = p.seq_offset + (uint32_t)s;
        const uint4 w = rng_words(p, seq, a.round, (uint32_t)pos, RNG_DRAFT, 0, 0);
        const double tgt = u24_to_double(w.x) * W;
        if (in_regs) {
            chunk = cdf.locate(tgt, lane, rem, refc);
        } else {
            chunk = cdf_locate<true>(part, p.NC, c, mc, true, lane, tot, tgt, rem);
            if (chunk >= 0) refc = __ldcg(part + chunk).x;
        }
    }
    uint4 vt[4], vx[4];
    load_lane_block<DT>(row, p.V, best, lane, vt);
    if (!FEATURES) load_lane_block<DT>(row, p.V, max(chunk, 0), lane, vx);

    // ---- features (Table 1): while the two chunks are on their way
    const float inv_T = FEATURES ? a.inv_T : p.inv_Tq;
    const double lw = log(W);
    const double m_s = (double)m * (double)inv_T;
    const double lse = m_s + lw;
    const double p1 = 1.0 / W;
    double H = lw - kLn2 * T2 / W;
    H = H > 0.0 ? H : 0.0;
    int cnt, first;
    float below;
    scan_top_block<DT>(vt, p.V, best, m, lane, cnt, first, below);
    const float m2 = (__popc(tie) >= 2 || cnt >= 2) ? m : fmaxf(fmaxf(other, c2all), below);
    const double p2 = (m2 > neg_inf()) ? exp(((double)m2 - (double)m) * (double)inv_T) / W : 0.0;

    if (FEATURES) {
        if (lane == 0) {
            float* fo = a.out_feat + (size_t)s * kFeat;
            fo[0] = (float)m_s; fo[1] = (float)lse; fo[2] = (float)p1; fo[3] = (float)p2; fo[4] = (float)H;
            fo[5] = (float)first;
        }
        return;
    }

    // ---- x_i ~ softmax(row) inside the chunk, from the weights the streaming pass summed
    int tok = -1;
    if (chunk >= 0) {
        const float kch = __fmul_rn(-refc, c);
        tok = pick_softmax_block<DT>(vx, p.V, chunk, c, kch, rem * exp2((double)kch + mc), lane);
    }
    if (lane == 0) {
        float* fo = st.feat + ((size_t)s * p.K + pos) * kFeat;
        fo[0] = (float)m_s; fo[1] = (float)lse; fo[2] = (float)p1; fo[3] = (float)p2; fo[4] = (float)H;
        fo[5] = (float)first;
        st.lse_q[(size_t)s * p.K + pos] = lse;
        const int arm = st.arm[(size_t)s * p.K + pos];
        bool stop = rule_stop(p, p.rule_of_arm[arm], p1, p2, H, st.sqrtH_prev[s], pos > 0, st.lambda[s]);
        st.sqrtH_prev[s] = sqrt(H);
        if (pos == p.K - 1) stop = true;
        st.n_drafted[s] = pos + 1;
        st.active[s] = stop ? 0 : 1;
        a.out_token[(size_t)s * a.tok_stride] = tok;
        a.out_continue[s] = stop ? 0 : 1;
        if (stop) {
            sc.stopped[atomicAdd(&sc.count[3], 1)] = s;
        } else {
            const int nslot = (a.slot + 1) % 3;
            sc.next_pos[s] = pos + 1;
            sc.list[(size_t)nslot * p.S + atomicAdd(&sc.count[nslot], 1)] = s;
        }
    }
}

// ============================================================================================
// One draft position (Algorithm 1, loop body) for every sequence still drafting.  Work item =
// (row, segment of the row); the persistent grid strides over the items.  Per item the CTA leaves a
// SegRec and, per 2 KB chunk, the chunk's partial softmax sum (for the inverse-CDF draw); a per-row
// counter tells the CTA that reduced the last segment to finish the row.  No CTA ever waits for
// another one.  FEATURES: rows 0 .. n_fixed-1 instead of the drafting list, features to out_feat.
// ============================================================================================
template <int DT, bool FEATURES>
__global__ void __launch_bounds__(kThreads, kResident)
k_draft_step(Params p, State st, Scratch sc, StepArgs a)
{
    constexpr int ESZ = Elem<DT>::BYTES;
    __shared__ WarpRec wrec[2][kWarps];
    __shared__ int todo[kTodo];              // rows whose last segment this CTA reduced: finished after the streaming
    __shared__ int n_todo;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) n_todo = 0;
    pdl_trigger();
    pdl_wait();
    const int n_rows = FEATURES ? a.n_fixed : sc.count[a.slot];
    const int32_t* list = sc.list + (size_t)a.slot * p.S;
    if (!FEATURES) {
        // the list two positions ahead is free again: nobody reads or appends to it during this launch
        if (blockIdx.x == 0 && tid == 0) sc.count[(a.slot + 2) % 3] = 0;
        // sequences that stopped at an earlier position draft nothing
        for (int s = blockIdx.x * kThreads + tid; s < p.S; s += gridDim.x * kThreads)
            if (sc.next_pos[s] < a.pos) { a.out_token[(size_t)s * a.tok_stride] = -1; a.out_continue[s] = 0; }
    }
    const int nseg = segments_for(p, n_rows, (int)gridDim.x);
    const int total = n_rows * nseg;
    const float c = a.c;

    int it = 0;
    for (int item = blockIdx.x; item < total; item += gridDim.x, ++it) {
        const int ai = item / nseg, g = item - ai * nseg;
        const int s = FEATURES ? ai : list[ai];
        const char* row = reinterpret_cast<const char*>(a.logits) + (size_t)s * a.row_stride * ESZ;
        const int c0 = (int)(((long long)g * p.NC) / nseg);
        const int c1 = (int)(((long long)(g + 1) * p.NC) / nseg);
        float2* part = sc.cdf + (size_t)s * p.NC;

        WarpAcc acc;
        acc.init();
        stream_chunks<DT, true, true>(acc, row, p.V, c0, c1, warp, lane, c,
                                      [&](int ch, float ref, float tot) { part[ch] = make_float2(ref, tot); });
        const float Sw = warp_sum_f(acc.S), Tw = warp_sum_f(acc.T);
        const int buf = it & 1;
        if (lane == 0) {
            WarpRec r;
            r.ref = acc.ref; r.k = acc.k; r.S = Sw; r.T = Tw; r.c1 = acc.c1; r.c2 = acc.c2; r.best = acc.best; r.pad = 0;
            wrec[buf][warp] = r;
        }
        __syncthreads();                     // also orders every warp's chunk partials before the fence below
        if (warp == (it & (kWarps - 1))) {   // the merging warp rotates; the others run ahead into the next item
            // lane w merges warp w's record: common reference = the largest, sums rescaled to it
            WarpRec r;
            r.ref = neg_inf(); r.k = 0.f; r.S = 0.f; r.T = 0.f; r.c1 = neg_inf(); r.c2 = neg_inf(); r.best = -1;
            if (lane < kWarps) r = wrec[buf][lane];
            const bool live = r.ref != neg_inf();                 // a NaN reference counts as live and poisons S
            const float ref = warp_max_f(r.ref);
            const float kref = __fmul_rn(-ref, c);
            const float dd = live ? kref - r.k : 0.f;             // <= 0
            const float f = live ? ex2_approx(dd) : 0.f;
            const float Sg = warp_sum_f(live ? f * r.S : 0.f);
            const float Tg = warp_sum_f(live ? f * fmaf(dd, r.S, r.T) : 0.f);
            // two largest chunk maxima of the segment (with multiplicity); lowest chunk holding the largest
            const unsigned tie = __ballot_sync(0xffffffffu, r.best >= 0 && r.c1 == ref);
            const int win = tie ? __ffs(tie) - 1 : 0;
            const float other = warp_max_f((lane == win) ? neg_inf() : r.c1);
            const float c2all = warp_max_f(r.c2);
            const float C2 = (__popc(tie) >= 2) ? ref : fmaxf(other, c2all);
            const int best = __reduce_min_sync(0xffffffffu, (tie >> lane) & 1u ? r.best : 0x7fffffff);
            int last = 0;
            if (lane == 0) {
                SegRec o;
                o.ref = ref; o.S = Sg; o.T = Tg; o.c2 = C2; o.best = (best == 0x7fffffff) ? -1 : best;
                o.pad0 = o.pad1 = o.pad2 = 0;
                store_segrec(sc.seg + (size_t)s * kMaxSeg + g, o);
                __threadfence();             // the segment (record and chunk partials) before it is counted
                last = atomicAdd(&sc.done[s], 1) == nseg - 1;
                if (last && n_todo < kTodo) { todo[n_todo] = s; n_todo = n_todo + 1; last = 0; }
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {                      // queue full: finish at once
                __threadfence();
                finish_row<DT, FEATURES>(p, st, sc, a, s, nseg, lane);
            }
        }
    }
    __syncthreads();
    // the rows this CTA completed, one warp each; their other segments were published before they were counted
    if (n_todo > 0) __threadfence();
    for (int j = warp; j < n_todo; j += kWarps) finish_row<DT, FEATURES>(p, st, sc, a, todo[j], nseg, lane);
}

// ============================================================================================
// Verification (Algorithm 1: verify, final token) as speculative sampling.  One cluster of CS CTAs
// per sequence, longest drafts first; CTA r streams the r-th slice of each target row.
// ============================================================================================
struct WalkArgs {
    const void* qlog; long long q_seq, q_pos;
    const void* plog; long long p_seq, p_pos;
    const int32_t* toks;
    int slot;                    // list of the sequences that were still drafting when verify was called
    uint32_t round;
    float cq, cp;
    int32_t* out_acc; int32_t* out_next;
};

struct WalkShared {
    float2 gather[2][kMaxCluster][kWarps];   // per-warp (reference, sum) of every CTA of the cluster, by row parity
    double ctot[2][kMaxCluster];             // per-CTA totals of the final draw: [0] residual, [1] target row
    float2 wrec[kWarps];
    double d0, d1;
    int i0, i1;
};

// Sends this warp's (ref, S) to every CTA of the cluster.
__device__ __forceinline__ void gather_send(cg::cluster_group& cl, WalkShared* sh, int par, int rank, int CS, int warp,
                                            int lane, float ref, float S) {
    if (lane < CS) {
        WalkShared* remote = cl.map_shared_rank(sh, lane);
        remote->gather[par][rank][warp] = make_float2(ref, S);
    }
}

// After the cluster barrier: row maximum and W = sum 2^((z-m)c) from the gathered records (warp 0, all lanes).
__device__ __forceinline__ void gather_reduce(const WalkShared* sh, int par, int CS, int lane, float c, float& m, double& W) {
    const int n = CS * kWarps;                       // <= 64: two records per lane
    const float2* g = &sh->gather[par][0][0];
    float2 r0 = make_float2(neg_inf(), 0.f), r1 = r0;
    if (lane < n) r0 = g[lane];
    if (lane + 32 < n) r1 = g[lane + 32];
    const bool bad = __any_sync(0xffffffffu, r0.x != r0.x || r0.y != r0.y || r1.x != r1.x || r1.y != r1.y);
    m = warp_max_f(fmaxf(r0.x, r1.x));
    const double mc = (double)m * (double)c;
    double w = 0.0;
    if (r0.x != neg_inf() && r0.y > 0.f) w += (double)r0.y * exp2(-((double)__fmul_rn(-r0.x, c) + mc));
    if (r1.x != neg_inf() && r1.y > 0.f) w += (double)r1.y * exp2(-((double)__fmul_rn(-r1.x, c) + mc));
    W = warp_sum_d(w);
    if (bad) W = (double)__int_as_float(0x7fc00000);
}

// Final draw, second half: the CTAs have exchanged their totals (ctot[which]); the CTA whose range holds
// u * total locates the chunk among its own partials and returns it (others return -1).  Whole warp 0.
// total <= 0 gives chunk -2 on every CTA.
template <bool SCALED>
__device__ __forceinline__ int owner_locate(const WalkShared* sh, int which, int rank, int CS, const float2* sm_part,
                                            int nloc, float c, double mc, double u, int lane, double& rem) {
    double mine = 0.0;
    if (lane < CS) mine = sh->ctot[which][lane];
    const double incl = warp_incl_scan_d(mine, lane);
    const double Z = __shfl_sync(0xffffffffu, incl, 31);
    rem = 0.0;
    if (!(Z > 0.0)) return -2;
    const double tgt = u * Z;
    const unsigned over = __ballot_sync(0xffffffffu, lane < CS && incl > tgt);
    const unsigned pos = __ballot_sync(0xffffffffu, lane < CS && mine > 0.0);
    const int owner = over ? __ffs(over) - 1 : 31 - __clz(pos);
    const double before = __shfl_sync(0xffffffffu, incl - mine, owner);
    if (rank != owner) return -1;
    const CdfTotals t = cdf_totals<false>(sm_part, nloc, c, mc, SCALED, lane);
    return cdf_locate<false>(sm_part, nloc, c, mc, SCALED, lane, t, tgt - before, rem);
}

template <int DT>
__global__ void __launch_bounds__(kThreads, kResident)
k_verify_walk(Params p, State st, Scratch sc, WalkArgs a)
{
    constexpr int ESZ = Elem<DT>::BYTES;
    extern __shared__ float2 sm_part[];                      // partial sums of this CTA's chunks
    __shared__ WalkShared sh;
    cg::cluster_group cl = cg::this_cluster();
    const int CS = (int)cl.num_blocks();
    const int rank = (int)cl.block_rank();
    const int cid = blockIdx.x / CS;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    pdl_trigger();
    pdl_wait();
    // longest drafts first: sequences still drafting, then the stopped ones, last stopped first
    const int n_act = sc.count[a.slot];
    const int s = (cid < n_act) ? sc.list[(size_t)a.slot * p.S + cid] : sc.stopped[p.S - 1 - cid];
    const int n = st.n_drafted[s];
    const uint32_t seq = p.seq_offset + (uint32_t)s;
    const char* pbase = reinterpret_cast<const char*>(a.plog) + (size_t)s * a.p_seq * ESZ;
    const char* qbase = reinterpret_cast<const char*>(a.qlog) + (size_t)s * a.q_seq * ESZ;
    const int c0 = (int)(((long long)rank * p.NC) / CS);
    const int c1 = (int)(((long long)(rank + 1) * p.NC) / CS);
    const int nloc = c1 - c0;
    const float cp = a.cp, cq = a.cq;

    // ---- walk: accept x_i iff u_i < p_i(x_i) / q_i(x_i)
    int acc_len = n;
    bool bad = false;
    float m_p = 0.f;
    double W_p = 0.0;
    for (int i = 0; i < n; ++i) {
        const char* prow = pbase + (size_t)i * a.p_pos * ESZ;
        WarpAcc acc;
        acc.init();
        stream_chunks<DT, false, false>(acc, prow, p.V, c0, c1, warp, lane, cp, [](int, float, float) {});
        const float Sw = warp_sum_f(acc.S);
        gather_send(cl, &sh, i & 1, rank, CS, warp, lane, acc.ref, Sw);
        cl.sync();
        if (warp == 0) {
            float m;
            double W;
            gather_reduce(&sh, i & 1, CS, lane, cp, m, W);
            int dec;
            if (!(m > neg_inf()) || !(m < CUDART_INF_F) || !(W > 0.0) || !(W < CUDART_INF)) {
                dec = -1;
            } else {
                const int x = a.toks[(size_t)s * p.K + i];
                if (x < 0 || x >= p.V) {
                    if (lane == 0 && rank == 0) atomicOr(&sc.status[0], 8ull);
                    dec = 0;
                } else {
                    const char* qrow = qbase + (size_t)i * a.q_pos * ESZ;
                    // p(x) / q(x) = exp((s_p(x) - m_p) - (s_q(x) - lse_q)) / W_p
                    const double dp = ((double)load_elem<DT>(prow, x) - (double)m) * (double)p.inv_Tp;
                    const double logq = (double)load_elem<DT>(qrow, x) * (double)p.inv_Tq - st.lse_q[(size_t)s * p.K + i];
                    const double ratio = exp(dp - logq) / W;
                    const uint4 w = rng_words(p, seq, a.round, (uint32_t)i, RNG_ACCEPT, 0, 0);
                    dec = (u24_to_double(w.x) < ratio) ? 1 : 0;
                }
            }
            if (lane == 0) { sh.i0 = dec; sh.d0 = (double)m; sh.d1 = W; }
        }
        __syncthreads();
        const int dec = sh.i0;
        m_p = (float)sh.d0;
        W_p = sh.d1;
        __syncthreads();
        if (dec != 1) { acc_len = i; bad = dec < 0; break; }
    }

    // ---- final token
    const uint4 w2 = rng_words(p, seq, a.round, (uint32_t)acc_len, RNG_RESAMPLE, 0, 0);
    const double u2 = u24_to_double(w2.x);
    const char* prow = pbase + (size_t)acc_len * a.p_pos * ESZ;
    int next = -1;                                            // meaningful on the CTA that draws the token
    bool mine = false;
    bool from_p = (acc_len == n) && !bad;
    if (!bad && acc_len < n) {
        // residual of the rejected slot: r = max(0, p - q), both rows in one pass (the target row is L2-hot)
        const char* qrow = qbase + (size_t)acc_len * a.q_pos * ESZ;
        const double lse_p = (double)m_p * (double)p.inv_Tp + log(W_p);
        const double lse_q = st.lse_q[(size_t)s * p.K + acc_len];
        const float kp = (float)(-lse_p * kLog2e), kq = (float)(-lse_q * kLog2e);
        const double dp = (double)kp + lse_p * kLog2e, dq = (double)kq + lse_q * kLog2e;   // rounding left in kp, kq
        const float beta = (float)exp2(dq - dp);            // p = 2^(zc+kp) 2^-dp,  q = 2^(zc+kq) 2^-dq
        for (int ch = c0 + warp; ch < c1; ch += kWarps) {
            uint4 vp[kVecPerLane], vq[kVecPerLane];
            load_chunk<DT>(prow, p.V, ch, lane, vp);
            load_chunk<DT>(qrow, p.V, ch, lane, vq);
            float r0 = 0.f, r1 = 0.f;
#pragma unroll
            for (int j = 0; j < kVecPerLane; ++j) {
                const uint32_t xp[4] = {vp[j].x, vp[j].y, vp[j].z, vp[j].w};
                const uint32_t xq[4] = {vq[j].x, vq[j].y, vq[j].z, vq[j].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (DT == DT_BF16) {
                        const float wp0 = ex2_approx(fmaf(__uint_as_float(xp[e] << 16), cp, kp));
                        const float wp1 = ex2_approx(fmaf(__uint_as_float(xp[e] & 0xffff0000u), cp, kp));
                        const float wq0 = ex2_approx(fmaf(__uint_as_float(xq[e] << 16), cq, kq));
                        const float wq1 = ex2_approx(fmaf(__uint_as_float(xq[e] & 0xffff0000u), cq, kq));
                        r0 += fmaxf(fmaf(wp0, beta, -wq0), 0.f);
                        r1 += fmaxf(fmaf(wp1, beta, -wq1), 0.f);
                    } else {
                        const float wp0 = ex2_approx(fmaf(__uint_as_float(xp[e]), cp, kp));
                        const float wq0 = ex2_approx(fmaf(__uint_as_float(xq[e]), cq, kq));
                        r0 += fmaxf(fmaf(wp0, beta, -wq0), 0.f);
                    }
                }
            }
            const float tot = warp_sum_f(r0 + r1);
            if (lane == 0) sm_part[ch - c0] = make_float2(0.f, tot);
        }
        __syncthreads();
        if (warp == 0) {
            const CdfTotals t = cdf_totals<false>(sm_part, nloc, 0.f, 0.0, false, lane);
            if (lane < CS) cl.map_shared_rank(&sh, lane)->ctot[0][rank] = t.W;
        }
        cl.sync();
        if (warp == 0) {
            double rem;
            const int lc = owner_locate<false>(&sh, 0, rank, CS, sm_part, nloc, 0.f, 0.0, u2, lane, rem);
            int tok = -1;
            if (lc >= 0) tok = pick_residual<DT>(prow, qrow, p.V, c0 + lc, cp, kp, cq, kq, beta, rem, lane);
            if (lane == 0) { sh.i0 = lc; sh.i1 = tok; }
        }
        __syncthreads();
        const int lc = sh.i0;
        if (lc == -2) {                                      // no residual mass (rounding only): draw from p instead
            from_p = true;
            if (tid == 0 && rank == 0) atomicOr(&sc.status[0], 4ull);
        } else if (lc >= 0) {
            mine = true;
            next = sh.i1;
        }
        __syncthreads();
    }
    if (from_p) {
        // bonus token (everything accepted), or the zero-residual fallback: draw from the target row
        const int par = acc_len & 1;                         // row acc_len - 1 (other parity) may still be read elsewhere
        WarpAcc acc;
        acc.init();
        stream_chunks<DT, false, true>(acc, prow, p.V, c0, c1, warp, lane, cp,
                                       [&](int ch, float ref, float tot) { sm_part[ch - c0] = make_float2(ref, tot); });
        const float Sw = warp_sum_f(acc.S);
        gather_send(cl, &sh, par, rank, CS, warp, lane, acc.ref, Sw);
        cl.sync();                                           // also orders sm_part for warp 0
        bool ok = false;
        double mc = 0.0;
        if (warp == 0) {
            float m;
            double W;
            gather_reduce(&sh, par, CS, lane, cp, m, W);
            ok = (m > neg_inf()) && (m < CUDART_INF_F) && (W > 0.0) && (W < CUDART_INF);
            mc = (double)m * (double)cp;
            double Wc = 0.0;
            if (ok) Wc = cdf_totals<false>(sm_part, nloc, cp, mc, true, lane).W;
            if (lane < CS) cl.map_shared_rank(&sh, lane)->ctot[1][rank] = Wc;
        }
        cl.sync();
        if (warp == 0) {
            int lc = -2, tok = -1;
            if (ok) {
                double rem;
                lc = owner_locate<true>(&sh, 1, rank, CS, sm_part, nloc, cp, mc, u2, lane, rem);
                if (lc >= 0) {
                    const float kch = __fmul_rn(-sm_part[lc].x, cp);
                    tok = pick_softmax<DT>(prow, p.V, c0 + lc, cp, kch, rem * exp2((double)kch + mc), lane);
                }
            }
            if (lane == 0) { sh.i0 = lc; sh.i1 = tok; }
        }
        __syncthreads();
        if (sh.i0 == -2) { bad = true; mine = false; next = -1; }
        else if (sh.i0 >= 0) { mine = true; next = sh.i1; }
    }
    if (tid == 0) {
        if (rank == 0) {
            if (bad) atomicOr(&sc.status[0], 2ull);
            st.accept_len[s] = acc_len;
            a.out_acc[s] = acc_len;
            if (bad) a.out_next[s] = -1;
            atomicAdd(&sc.status[2], (unsigned long long)(acc_len + 1));
            if (acc_len < n) atomicAdd(&sc.status[3], 1ull);
        }
        if (mine && !bad) a.out_next[s] = next;
    }
}

// ============================================================================================
// Bandit arm for one slot (sequence level: slot 0; token level: slot = draft position), Section 3.3.
// Whole warp; every lane returns the arm.
// ============================================================================================
__device__ __forceinline__ int select_arm(const Params& p, const State& st, int s, int slot, uint32_t round,
                                          uint32_t* hist, int lane) {
    const size_t o = ((size_t)s * p.P + slot) * p.A;
    const uint32_t seq = p.seq_offset + (uint32_t)s;
    if (p.policy == 1 && p.level == 1)
        return ts_beta_select_warp(p, st.cnt + o, st.rsum + o, seq, round, (uint32_t)slot, hist, lane);
    int arm = 0;
    if (lane == 0) {
        if (p.policy == 0) arm = ucb1_select(st.cnt + o, st.rsum + o, p.A, p.ucb_c2);
        else if (p.policy == 2) arm = ucb_tuned_select(st.cnt + o, st.rsum + o, st.rsum2 + o, p.A);
        else arm = ts_gauss_select(p, st.cnt + o, st.rsum + o, seq, round, 0u);
    }
    return __shfl_sync(0xffffffffu, arm, 0);
}

// Arms of round `round` for every sequence and slot, and the round's bookkeeping (one warp per sequence).
__device__ __forceinline__ void begin_round(const Params& p, const State& st, const Scratch& sc, int s, uint32_t round,
                                            uint32_t* hist, int lane) {
    if (p.level == 0) {
        const int arm = select_arm(p, st, s, 0, round, hist, lane);
        for (int k = lane; k < p.K; k += 32) st.arm[(size_t)s * p.K + k] = arm;
    } else if (p.policy == 1) {
        for (int k = 0; k < p.K; ++k) {
            const int arm = select_arm(p, st, s, k, round, hist, lane);
            if (lane == 0) st.arm[(size_t)s * p.K + k] = arm;
        }
    } else {
        // one lane per position; select_arm's scalar branch runs on lane 0 only, so call the scalar code directly
        for (int k = lane; k < p.K; k += 32) {
            const size_t o = ((size_t)s * p.P + k) * p.A;
            st.arm[(size_t)s * p.K + k] = (p.policy == 0) ? ucb1_select(st.cnt + o, st.rsum + o, p.A, p.ucb_c2)
                                                          : ucb_tuned_select(st.cnt + o, st.rsum + o, st.rsum2 + o, p.A);
        }
    }
    if (lane == 0) {
        st.active[s] = 1; st.n_drafted[s] = 0; st.sqrtH_prev[s] = 0.0;
        sc.list[s] = s; sc.next_pos[s] = 0; sc.done[s] = 0;
        if (s == 0) { sc.count[0] = p.S; sc.count[1] = 0; sc.count[2] = 0; sc.count[3] = 0; }
    }
}

// update(pi, |Y|, |X|, gamma): rewards, arm statistics, AdaEDL; then the arms of the next round.
__global__ void __launch_bounds__(128)
k_update(Params p, State st, Scratch sc, uint32_t next_round)
{
    __shared__ uint32_t hist[4][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x * 4 + warp;
    pdl_trigger();
    pdl_wait();
    if (s >= p.S) return;
    if (lane == 0) {
        const int n = st.n_drafted[s], a = st.accept_len[s];
        double r_out = 0.0;
        if (n > 0) {
            if (p.level == 0) {
                const double r = p.reward_kind ? ((double)a / (double)p.K)
                                               : (p.reward_alpha * ((double)a / (double)p.K) +
                                                  (1.0 - p.reward_alpha) * ((double)a / (double)n));
                const size_t o = (size_t)s * p.A + st.arm[(size_t)s * p.K];
                st.cnt[o] += 1; st.rsum[o] += r; st.rsum2[o] += r * r;
                r_out = r;
            } else {
                const int last = p.token_update_all ? n : min(a + 1, n);
                for (int i = 0; i < last; ++i) {
                    const double r = (i < a) ? 1.0 : 0.0;
                    const size_t o = ((size_t)s * p.K + i) * p.A + st.arm[(size_t)s * p.K + i];
                    st.cnt[o] += 1; st.rsum[o] += r; st.rsum2[o] += r * r;
                }
                r_out = (double)a;
            }
            // AdaEDL, as printed: lambda <- b2*lambda + (1-b2)*(lambda + eps*sign(alpha - r))
            const double r = (double)a / (double)n;
            const double d = p.ada_alpha - r;
            const double sgn = (double)((d > 0.0) - (d < 0.0));
            st.acc_rate[s] = p.ada_beta1 * st.acc_rate[s] + (1.0 - p.ada_beta1) * r;
            st.lambda[s] = p.ada_beta2 * st.lambda[s] + (1.0 - p.ada_beta2) * (st.lambda[s] + p.ada_eps * sgn);
        }
        st.reward[s] = r_out;
    }
    __syncwarp();
    begin_round(p, st, sc, s, next_round, hist[warp], lane);
}

// Start of a round without an update before it (a new handle, a changed parameter, restored state):
// arms and bookkeeping only.
__global__ void __launch_bounds__(128)
k_begin_round(Params p, State st, Scratch sc, uint32_t round, int reset_adaedl)
{
    __shared__ uint32_t hist[4][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x * 4 + warp;
    pdl_trigger();
    pdl_wait();
    if (s >= p.S) return;
    if (reset_adaedl && lane == 0) { st.lambda[s] = p.ada_lambda0; st.acc_rate[s] = p.ada_acc0; }
    __syncwarp();
    begin_round(p, st, sc, s, round, hist[warp], lane);
}

// After tapout_set_state in the middle of a round: the drafting list of position `pos` and the list of
// stopped sequences (shortest drafts first, a counting sort) are rebuilt from the active flags and the
// drafted lengths.  Single CTA; the order inside a list only affects scheduling.
__global__ void __launch_bounds__(1024)
k_rebuild_lists(Params p, State st, Scratch sc, int pos)
{
    __shared__ int hist[1026];
    __shared__ int sh_n;
    const int tid = threadIdx.x;
    const int slot = pos % 3;
    for (int i = tid; i <= p.K + 1; i += blockDim.x) hist[i] = 0;
    if (tid == 0) sh_n = 0;
    __syncthreads();
    for (int s = tid; s < p.S; s += blockDim.x) {
        sc.done[s] = 0;
        if (st.active[s]) {
            sc.next_pos[s] = pos;
            sc.list[(size_t)slot * p.S + atomicAdd(&sh_n, 1)] = s;
        } else {
            sc.next_pos[s] = -1;
            atomicAdd(&hist[min(max(st.n_drafted[s], 0), p.K)], 1);
        }
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int n = 0; n <= p.K; ++n) { const int h = hist[n]; hist[n] = run; run += h; }
        sc.count[3] = run;
        sc.count[slot] = sh_n;
        sc.count[(slot + 1) % 3] = 0;
        sc.count[(slot + 2) % 3] = 0;
    }
    __syncthreads();
    for (int s = tid; s < p.S; s += blockDim.x)
        if (!st.active[s]) sc.stopped[atomicAdd(&hist[min(max(st.n_drafted[s], 0), p.K)], 1)] = s;
}

}  // namespace tpo
