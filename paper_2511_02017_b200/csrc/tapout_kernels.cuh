// Kernels of libtapout (sm_100a).  Streaming kernels read each needed logit row from HBM exactly
// once with 128-bit coalesced loads; everything per-row that is scalar runs in double.
#pragma once

#include "tapout_device.cuh"

namespace tpo {

struct WarpRec { float ref, k, S, T, c1, c2; int best; int pad; };

// How many CTAs share one draft row, decided on the device from the number of rows actually drafted at
// this position (the host never learns it): enough items for about six per CTA, at least one chunk per
// warp, at most kMaxSeg.  The streaming pass and its finish kernel must agree, hence one function.
__device__ __forceinline__ int segments_for(const Params& p, int n_rows, int grid) {
    if (p.nseg > 0) return p.nseg;
    int nseg = (6 * grid + n_rows - 1) / max(n_rows, 1);
    nseg = min(nseg, max(p.NC / kWarps, 1));
    return max(1, min(nseg, min(kMaxSeg, p.NC)));
}

// ============================================================================================
// Draft rows, streaming pass.  Work item = (sequence still drafting, segment of its row); a
// persistent grid strides over the items.  Per item the CTA leaves a SegRec and, per 2 KB chunk,
// the chunk's partial softmax sum (for the inverse-CDF draw in the finish kernel).  Each warp keeps
// the next chunk's loads in flight while it folds the current one.
// ============================================================================================
template <int DT>
__global__ void __launch_bounds__(kThreads, 3)
k_draft_rows(Params p, Scratch sc, const void* __restrict__ logits, long long row_stride, int parity,
             int n_fixed, int grid_ref, float c)
{
    __shared__ WarpRec wrec[kWarps];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_rows = (n_fixed >= 0) ? n_fixed : sc.count[parity];
    if (n_fixed < 0 && blockIdx.x == 0 && tid == 0) sc.count[parity ^ 1] = 0;   // this step's finish appends to it
    const int32_t* list = sc.list + (size_t)parity * p.S;
    const int nseg = segments_for(p, n_rows, grid_ref);
    const int total = n_rows * nseg;

    for (int item = blockIdx.x; item < total; item += gridDim.x) {
        const int ai = item / nseg, g = item - ai * nseg;
        const int s = (n_fixed >= 0) ? ai : list[ai];
        const char* row = reinterpret_cast<const char*>(logits) + (size_t)s * row_stride * Elem<DT>::BYTES;
        const int c0 = (int)(((long long)g * p.NC) / nseg);
        const int c1 = (int)(((long long)(g + 1) * p.NC) / nseg);
        float2* part = sc.cdf + (size_t)s * p.NC;

        WarpAcc acc;
        acc.init();
        int ch = c0 + warp;
        uint4 cur[kVecPerLane], nxt[kVecPerLane];
        if (ch < c1) load_chunk<DT>(row, p.V, ch, lane, cur);
        while (ch < c1) {
            const int chn = ch + kWarps;
            if (chn < c1) load_chunk<DT>(row, p.V, chn, lane, nxt);
            const float tot = fold_chunk<DT, true, true>(acc, cur, ch, c);
            if (lane == 0) part[ch] = make_float2(acc.ref, tot);
#pragma unroll
            for (int j = 0; j < kVecPerLane; ++j) cur[j] = nxt[j];
            ch = chn;
        }
        const float Sw = warp_sum_f(acc.S), Tw = warp_sum_f(acc.T);
        if (lane == 0) {
            WarpRec r;
            r.ref = acc.ref; r.k = acc.k; r.S = Sw; r.T = Tw; r.c1 = acc.c1; r.c2 = acc.c2; r.best = acc.best; r.pad = 0;
            wrec[warp] = r;
        }
        __syncthreads();
        if (warp == 0) {
            // lane w merges warp w's record: common reference = the largest, sums rescaled to it
            WarpRec r;
            r.ref = neg_inf(); r.k = 0.f; r.S = 0.f; r.T = 0.f; r.c1 = neg_inf(); r.c2 = neg_inf(); r.best = -1;
            if (lane < kWarps) r = wrec[lane];
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
            if (lane == 0) {
                SegRec o;
                o.ref = ref; o.S = Sg; o.T = Tg; o.c2 = C2; o.best = (best == 0x7fffffff) ? -1 : best;
                o.pad0 = o.pad1 = o.pad2 = 0;
                sc.seg[(size_t)s * kMaxSeg + g] = o;
            }
        }
        __syncthreads();
    }
}

// Row-level result of combining the segments of one row (whole warp; every lane holds the same values).
struct RowComb {
    bool valid;
    float m, m2;         // raw maximum and second largest logit
    int argmax;
    double mc;           // m * c
    double W, T2;        // sum of 2^((z-m)c) ; sum of w * t (log2 units)
    CdfTotals tot;
};

template <int DT>
__device__ __forceinline__ RowComb combine_row(const Params& p, const Scratch& sc, const void* row, int s, int nseg,
                                               float c, int lane) {
    RowComb rc;
    SegRec r;
    r.ref = neg_inf(); r.S = 0.f; r.T = 0.f; r.c2 = neg_inf(); r.best = -1;
    if (lane < nseg) r = sc.seg[(size_t)s * kMaxSeg + lane];
    const bool has_nan = __any_sync(0xffffffffu, (r.S != r.S) || (r.T != r.T) || (r.ref != r.ref));
    const float m = warp_max_f(r.ref);
    rc.m = m;
    rc.mc = (double)m * (double)c;
    double Tg = 0.0;
    if (lane < nseg && r.ref > neg_inf() && r.ref < CUDART_INF_F) {
        const double d = (double)__fmul_rn(-r.ref, c) + rc.mc;           // >= 0 up to rounding
        Tg = exp2(-d) * ((double)r.T - d * (double)r.S);
    }
    rc.T2 = warp_sum_d(Tg);
    rc.tot = cdf_totals(sc.cdf + (size_t)s * p.NC, p.NC, c, rc.mc, true, lane);
    rc.W = rc.tot.W;
    rc.valid = !has_nan && (m > neg_inf()) && (m < CUDART_INF_F) && (rc.W > 0.0) && (rc.W < CUDART_INF);
    rc.m2 = neg_inf();
    rc.argmax = -1;
    if (rc.valid) {
        // second largest element and argmax: only the (lowest) chunk holding the maximum needs a second look
        const unsigned tie = __ballot_sync(0xffffffffu, lane < nseg && r.ref == m);
        const int win = __ffs(tie) - 1;
        const float other = warp_max_f((lane == win || lane >= nseg) ? neg_inf() : r.ref);
        const float c2all = warp_max_f(r.c2);
        const int best = __shfl_sync(0xffffffffu, r.best, win);
        int cnt, first;
        float below;
        scan_top_chunk<DT>(row, p.V, best, m, lane, cnt, first, below);
        rc.argmax = first;
        rc.m2 = (__popc(tie) >= 2 || cnt >= 2) ? m : fmaxf(fmaxf(other, c2all), below);
    }
    return rc;
}

struct RowFeat { double m_s, lse, p1, p2, H; };

__device__ __forceinline__ RowFeat features_of(const RowComb& rc, float inv_T) {
    RowFeat f;
    const double lw = log(rc.W);
    f.m_s = (double)rc.m * (double)inv_T;
    f.lse = f.m_s + lw;
    f.p1 = 1.0 / rc.W;
    f.p2 = (rc.m2 > neg_inf()) ? exp(((double)rc.m2 - (double)rc.m) * (double)inv_T) / rc.W : 0.0;
    double H = lw - kLn2 * rc.T2 / rc.W;
    f.H = H > 0.0 ? H : 0.0;
    return f;
}

// ============================================================================================
// Draft rows, finish: one warp per sequence.  Arm selection, features, token draw, stop rule,
// bookkeeping, next active list.
// ============================================================================================
template <int DT>
__global__ void __launch_bounds__(128)
k_draft_finish(Params p, State st, Scratch sc, const void* __restrict__ logits, long long row_stride, int pos,
               int parity, uint32_t round, int grid_ref, float c, int32_t* __restrict__ out_token,
               long long tok_stride, uint8_t* __restrict__ out_continue)
{
    __shared__ uint32_t hist[4][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x * 4 + warp;
    if (s >= p.S) return;
    if (!st.active[s]) {
        if (lane == 0) { out_token[(size_t)s * tok_stride] = -1; out_continue[s] = 0; }
        return;
    }
    const uint32_t seq = p.seq_offset + (uint32_t)s;

    // ---- which arm is consulted at this position
    int arm = 0;
    if (p.level == 0 && pos > 0) {
        arm = st.arm[(size_t)s * p.K];
    } else {
        const int slot = (p.level == 0) ? 0 : pos;
        const size_t o = ((size_t)s * p.P + slot) * p.A;
        if (p.policy == 1 && p.level == 1) {
            arm = ts_beta_select_warp(p, st.cnt + o, st.rsum + o, seq, round, (uint32_t)pos, hist[warp], lane);
        } else {
            if (lane == 0) {
                if (p.policy == 0) arm = ucb1_select(st.cnt + o, st.rsum + o, p.A, p.ucb_c2);
                else if (p.policy == 2) arm = ucb_tuned_select(st.cnt + o, st.rsum + o, st.rsum2 + o, p.A);
                else arm = ts_gauss_select(p, st.cnt + o, st.rsum + o, seq, round, 0u);
            }
            arm = __shfl_sync(0xffffffffu, arm, 0);
        }
        if (p.level == 0) { for (int k = lane; k < p.K; k += 32) st.arm[(size_t)s * p.K + k] = arm; }
        else if (lane == 0) st.arm[(size_t)s * p.K + pos] = arm;
    }

    const char* row = reinterpret_cast<const char*>(logits) + (size_t)s * row_stride * Elem<DT>::BYTES;
    const int nseg = segments_for(p, sc.count[parity], grid_ref);
    const RowComb rc = combine_row<DT>(p, sc, row, s, nseg, c, lane);
    if (lane == 0) atomicAdd(&sc.status[1], 1ull);
    if (!rc.valid) {
        if (lane == 0) {
            atomicOr(&sc.status[0], 1ull);
            out_token[(size_t)s * tok_stride] = -1; out_continue[s] = 0; st.active[s] = 0;
        }
        return;
    }
    const RowFeat f = features_of(rc, p.inv_Tq);

    // ---- x_i ~ softmax(row): chunk by the partial sums, token inside the chunk in double
    const uint4 w = rng_words(p, seq, round, (uint32_t)pos, RNG_DRAFT, 0, 0);
    const double u = u24_to_double(w.x);
    double rem;
    const int chunk = cdf_locate(sc.cdf + (size_t)s * p.NC, p.NC, c, rc.mc, true, lane, rc.tot, u * rc.W, rem);
    RegWeights<chunk_elems<DT>() / 32> wreg;
    const int tok = pick_softmax<DT>(wreg, row, p.V, chunk, rem, (double)p.inv_Tq, f.m_s, lane);

    if (lane == 0) {
        float* fo = st.feat + ((size_t)s * p.K + pos) * kFeat;
        fo[0] = (float)f.m_s; fo[1] = (float)f.lse; fo[2] = (float)f.p1; fo[3] = (float)f.p2; fo[4] = (float)f.H;
        fo[5] = (float)rc.argmax;
        st.lse_q[(size_t)s * p.K + pos] = f.lse;
        bool stop = rule_stop(p, p.rule_of_arm[arm], f.p1, f.p2, f.H, st.sqrtH_prev[s], pos > 0, st.lambda[s]);
        st.sqrtH_prev[s] = sqrt(f.H);
        if (pos == p.K - 1) stop = true;
        st.n_drafted[s] = pos + 1;
        st.active[s] = stop ? 0 : 1;
        out_token[(size_t)s * tok_stride] = tok;
        out_continue[s] = stop ? 0 : 1;
        if (!stop) {
            const int slot = atomicAdd(&sc.count[parity ^ 1], 1);
            sc.list[(size_t)(parity ^ 1) * p.S + slot] = s;
        }
    }
}

// Features only (tapout_row_stats): one warp per row.
template <int DT>
__global__ void __launch_bounds__(128)
k_rows_features(Params p, Scratch sc, const void* __restrict__ logits, long long row_stride, int n_rows, int grid_ref,
                float c, float inv_T, float* __restrict__ out)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x * 4 + warp;
    if (s >= n_rows) return;
    const char* row = reinterpret_cast<const char*>(logits) + (size_t)s * row_stride * Elem<DT>::BYTES;
    const RowComb rc = combine_row<DT>(p, sc, row, s, segments_for(p, n_rows, grid_ref), c, lane);
    if (lane != 0) return;
    float* fo = out + (size_t)s * kFeat;
    if (!rc.valid) {
        const float qn = __int_as_float(0x7fc00000);
        fo[0] = fo[1] = fo[2] = fo[3] = fo[4] = qn; fo[5] = -1.f;
        return;
    }
    const RowFeat f = features_of(rc, inv_T);
    fo[0] = (float)f.m_s; fo[1] = (float)f.lse; fo[2] = (float)f.p1; fo[3] = (float)f.p2; fo[4] = (float)f.H;
    fo[5] = (float)rc.argmax;
}

// ============================================================================================
// Verification.  Sequences are taken longest-draft-first from a queue; one CTA walks one
// sequence's target rows, stops at the first rejection, then draws the residual or bonus token.
// ============================================================================================
__global__ void __launch_bounds__(1024)
k_verify_prepare(Params p, State st, Scratch sc)
{
    __shared__ int hist[1026];
    const int tid = threadIdx.x;
    for (int i = tid; i <= p.K + 1; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int s = tid; s < p.S; s += blockDim.x) atomicAdd(&hist[st.n_drafted[s]], 1);
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int n = p.K; n >= 0; --n) { const int h = hist[n]; hist[n] = run; run += h; }
        sc.count[2] = 0;
    }
    __syncthreads();
    for (int s = tid; s < p.S; s += blockDim.x) {
        const int slot = atomicAdd(&hist[st.n_drafted[s]], 1);
        sc.order[slot] = s;
    }
}

// Token picks of the verify kernel, kept out of line so that their double-precision exponentials do not
// set the register budget of the streaming loops around them.
template <int DT>
__device__ __noinline__ int pick_softmax_smem(double* sm_w, const void* row, int V, int chunk, double rem,
                                              double inv_T, double m_s, int lane) {
    SmemWeights<chunk_elems<DT>() / 32> w{sm_w, lane};
    return pick_softmax<DT>(w, row, V, chunk, rem, inv_T, m_s, lane);
}

template <int DT>
__device__ __noinline__ int pick_residual_smem(double* sm_w, const void* prow, const void* qrow, int V, int chunk,
                                               double rem, double iTp, double lse_p, double iTq, double lse_q,
                                               int lane) {
    SmemWeights<chunk_elems<DT>() / 32> w{sm_w, lane};
    return pick_residual<DT>(w, prow, qrow, V, chunk, rem, iTp, lse_p, iTq, lse_q, lane);
}

// Softmax normaliser of one row by the whole CTA.  Every thread returns the raw maximum m and
// W = sum 2^((z-m)c).  With PART the per-chunk partial sums go to sm_part (for the bonus draw).
template <int DT, bool PART>
__device__ __forceinline__ void block_lse(const void* row, int V, int NC, float c, float2* sm_part, float2* wrec,
                                          float& m, double& W)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WarpAcc acc;
    acc.init();
    for (int ch = warp; ch < NC; ch += kWarps) {
        uint4 v[kVecPerLane];
        load_chunk<DT>(row, V, ch, lane, v);
        const float tot = fold_chunk<DT, false, PART>(acc, v, ch, c);
        if (PART && lane == 0) sm_part[ch] = make_float2(acc.ref, tot);
    }
    const float S = warp_sum_f(acc.S);
    if (lane == 0) wrec[warp] = make_float2(acc.ref, S);
    __syncthreads();
    float mm = neg_inf();
    bool bad = false;
    for (int w = 0; w < kWarps; ++w) {
        const float2 r = wrec[w];
        if (r.x != r.x || r.y != r.y) bad = true;
        mm = fmaxf(mm, r.x);
    }
    const double mc = (double)mm * (double)c;
    double Wd = 0.0;
    for (int w = 0; w < kWarps; ++w) {
        const float2 r = wrec[w];
        if (r.x == neg_inf() || !(r.y > 0.f)) continue;
        Wd += (double)r.y * exp2(-((double)__fmul_rn(-r.x, c) + mc));
    }
    if (bad) Wd = (double)__int_as_float(0x7fc00000);
    m = mm;
    W = Wd;
    __syncthreads();
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 3)
k_verify_walk(Params p, State st, Scratch sc, const void* __restrict__ qlog, long long q_seq, long long q_pos,
              const void* __restrict__ plog, long long p_seq, long long p_pos, const int32_t* __restrict__ toks,
              uint32_t round, float cq, float cp, int32_t* __restrict__ out_acc, int32_t* __restrict__ out_next)
{
    constexpr int ESZ = Elem<DT>::BYTES;
    extern __shared__ double sm_dyn[];                       // [chunk_elems] pick weights, then [NC] chunk partials
    double* sm_w = sm_dyn;
    float2* sm_part = reinterpret_cast<float2*>(sm_dyn + chunk_elems<DT>());
    __shared__ float2 wrec[kWarps];
    __shared__ int sh_i, sh_dec, sh_tok;
    __shared__ double sh_lse;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    for (;;) {
        __syncthreads();
        if (tid == 0) sh_i = atomicAdd(&sc.count[2], 1);
        __syncthreads();
        const int qi = sh_i;
        if (qi >= p.S) break;
        const int s = sc.order[qi];
        const int n = st.n_drafted[s];
        const uint32_t seq = p.seq_offset + (uint32_t)s;
        const char* pbase = reinterpret_cast<const char*>(plog) + (size_t)s * p_seq * ESZ;
        const char* qbase = reinterpret_cast<const char*>(qlog) + (size_t)s * q_seq * ESZ;

        // ---- walk: accept x_i iff u_i < p_i(x_i) / q_i(x_i)
        int a = n;
        bool bad = false;
        float m_p = 0.f;
        double W_p = 0.0, lse_p = 0.0;
        for (int i = 0; i < n; ++i) {
            const char* prow = pbase + (size_t)i * p_pos * ESZ;
            block_lse<DT, false>(prow, p.V, p.NC, cp, nullptr, wrec, m_p, W_p);
            if (tid == 0) {
                int dec;
                if (!(m_p > neg_inf()) || !(m_p < CUDART_INF_F) || !(W_p > 0.0) || !(W_p < CUDART_INF)) {
                    dec = -1;
                } else {
                    const double lse = (double)m_p * (double)p.inv_Tp + log(W_p);
                    sh_lse = lse;
                    const int x = toks[(size_t)s * p.K + i];
                    if (x < 0 || x >= p.V) {
                        atomicOr(&sc.status[0], 8ull);
                        dec = 0;
                    } else {
                        const char* qrow = qbase + (size_t)i * q_pos * ESZ;
                        const double logp = (double)load_elem<DT>(prow, x) * (double)p.inv_Tp - lse;
                        const double logq = (double)load_elem<DT>(qrow, x) * (double)p.inv_Tq - st.lse_q[(size_t)s * p.K + i];
                        const double ratio = exp(logp - logq);
                        const uint4 w = rng_words(p, seq, round, (uint32_t)i, RNG_ACCEPT, 0, 0);
                        dec = (u24_to_double(w.x) < ratio) ? 1 : 0;
                    }
                }
                sh_dec = dec;
            }
            __syncthreads();
            const int dec = sh_dec;
            lse_p = sh_lse;
            __syncthreads();
            if (dec != 1) { a = i; bad = dec < 0; break; }
        }

        // ---- final token
        const uint4 w2 = rng_words(p, seq, round, (uint32_t)a, RNG_RESAMPLE, 0, 0);
        const double u2 = u24_to_double(w2.x);
        const char* prow = pbase + (size_t)a * p_pos * ESZ;
        int next = -1;
        bool from_p = (a == n) && !bad;
        if (!bad && a < n) {
            // residual of the rejected slot: r = max(0, p - q), both rows in one pass
            const char* qrow = qbase + (size_t)a * q_pos * ESZ;
            const double lse_q = st.lse_q[(size_t)s * p.K + a];
            const float kp = (float)(-lse_p * kLog2e), kq = (float)(-lse_q * kLog2e);
            const double dp = (double)kp + lse_p * kLog2e, dq = (double)kq + lse_q * kLog2e;   // rounding left in kp, kq
            const float beta = (float)exp2(dq - dp);        // p = 2^(zc+kp) 2^-dp,  q = 2^(zc+kq) 2^-dq
            for (int ch = warp; ch < p.NC; ch += kWarps) {
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
                if (lane == 0) sm_part[ch] = make_float2(0.f, tot);
            }
            __syncthreads();
            if (warp == 0) {
                const CdfTotals t = cdf_totals(sm_part, p.NC, 0.f, 0.0, false, lane);
                int tok = -2;                                  // -2: no residual mass
                if (t.W > 0.0) {
                    double rem;
                    const int chunk = cdf_locate(sm_part, p.NC, 0.f, 0.0, false, lane, t, u2 * t.W, rem);
                    tok = pick_residual_smem<DT>(sm_w, prow, qrow, p.V, chunk, rem * exp2(-dq), (double)p.inv_Tp,
                                                 lse_p, (double)p.inv_Tq, lse_q, lane);
                }
                if (lane == 0) sh_tok = tok;
            }
            __syncthreads();
            next = sh_tok;
            if (next == -2) {
                from_p = true;
                if (tid == 0) atomicOr(&sc.status[0], 4ull);
            }
            __syncthreads();
        }
        if (from_p) {
            // bonus token (everything accepted), or the zero-residual fallback: draw from the target row
            block_lse<DT, true>(prow, p.V, p.NC, cp, sm_part, wrec, m_p, W_p);
            const bool ok = (m_p > neg_inf()) && (m_p < CUDART_INF_F) && (W_p > 0.0) && (W_p < CUDART_INF);
            if (!ok) {
                bad = true;
                next = -1;
            } else {
                if (warp == 0) {
                    const double mc = (double)m_p * (double)cp;
                    const CdfTotals t = cdf_totals(sm_part, p.NC, cp, mc, true, lane);
                    double rem;
                    const int chunk = cdf_locate(sm_part, p.NC, cp, mc, true, lane, t, u2 * t.W, rem);
                    const int tok = pick_softmax_smem<DT>(sm_w, prow, p.V, chunk, rem, (double)p.inv_Tp,
                                                          (double)m_p * (double)p.inv_Tp, lane);
                    if (lane == 0) sh_tok = tok;
                }
                __syncthreads();
                next = sh_tok;
            }
        }
        if (tid == 0) {
            if (bad) atomicOr(&sc.status[0], 2ull);
            st.accept_len[s] = a;
            out_acc[s] = a;
            out_next[s] = next;
            atomicAdd(&sc.status[2], (unsigned long long)(a + 1));
            if (a < n) atomicAdd(&sc.status[3], 1ull);
        }
    }
}

// ============================================================================================
// update(pi, |Y|, |X|, gamma): rewards, arm statistics, AdaEDL; then the next round's bookkeeping.
// ============================================================================================
__global__ void __launch_bounds__(256)
k_update(Params p, State st, Scratch sc)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= p.S) return;
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
    st.active[s] = 1; st.n_drafted[s] = 0; st.sqrtH_prev[s] = 0.0;
    sc.list[s] = s;
    if (s == 0) { sc.count[0] = p.S; sc.count[1] = 0; }
}

// Start-of-life (and after a parameter that re-initialises AdaEDL): round bookkeeping only.
__global__ void __launch_bounds__(256)
k_reset_round(Params p, State st, Scratch sc, int reset_adaedl)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= p.S) return;
    if (reset_adaedl) { st.lambda[s] = p.ada_lambda0; st.acc_rate[s] = p.ada_acc0; }
    st.active[s] = 1; st.n_drafted[s] = 0; st.sqrtH_prev[s] = 0.0;
    sc.list[s] = s;
    if (s == 0) { sc.count[0] = p.S; sc.count[1] = 0; }
}

// After tapout_set_state in the middle of a round: the list of drafting sequences for the next
// position is rebuilt from the active flags (single CTA, order by sequence id).
__global__ void __launch_bounds__(1024)
k_rebuild_active(Params p, State st, Scratch sc, int parity)
{
    __shared__ int sh_n;
    if (threadIdx.x == 0) sh_n = 0;
    __syncthreads();
    for (int s = threadIdx.x; s < p.S; s += blockDim.x)
        if (st.active[s]) sc.list[(size_t)parity * p.S + atomicAdd(&sh_n, 1)] = s;
    __syncthreads();
    if (threadIdx.x == 0) sc.count[parity] = sh_n;
}

}  // namespace tpo
