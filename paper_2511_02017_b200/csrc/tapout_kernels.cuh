// Kernels of libtapout (sm_100a).  Streaming kernels read each needed logit row from HBM exactly
// once with 128-bit coalesced loads; everything per-row that is scalar runs in double.
#pragma once

#include "tapout_device.cuh"

namespace tpo {

struct WarpRec { float ref, k, S, T, c1, c2; int best; int pad; };

// ============================================================================================
// Draft rows, streaming pass.  Work item = (sequence still drafting, segment of its row); a
// persistent grid strides over the items.  Per item the CTA leaves a SegRec and, per 2 KB chunk,
// the chunk's partial softmax sum (for the inverse-CDF draw in the finish kernel).
// ============================================================================================
template <int DT>
__global__ void __launch_bounds__(kThreads, 4)
k_draft_rows(Params p, Scratch sc, const void* __restrict__ logits, long long row_stride, int parity,
             int n_fixed, float c)
{
    constexpr int CH = chunk_elems<DT>();
    __shared__ WarpRec wrec[kWarps];
    __shared__ float sh_C1, sh_C2;
    __shared__ int sh_best, sh_cnt, sh_first, sh_below;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_rows = (n_fixed >= 0) ? n_fixed : sc.count[parity];
    if (n_fixed < 0 && blockIdx.x == 0 && tid == 0) sc.count[parity ^ 1] = 0;   // this step's finish appends to it
    const int32_t* list = sc.list + (size_t)parity * p.S;
    const int total = n_rows * p.nseg;

    for (int item = blockIdx.x; item < total; item += gridDim.x) {
        const int ai = item / p.nseg, g = item - ai * p.nseg;
        const int s = (n_fixed >= 0) ? ai : list[ai];
        const char* row = reinterpret_cast<const char*>(logits) + (size_t)s * row_stride * Elem<DT>::BYTES;
        const int c0 = (int)(((long long)g * p.NC) / p.nseg);
        const int c1 = (int)(((long long)(g + 1) * p.NC) / p.nseg);
        float2* part = sc.cdf + (size_t)s * p.NC;

        WarpAcc acc;
        acc.init();
        for (int ch = c0 + warp; ch < c1; ch += kWarps) {
            uint4 v[kVecPerLane];
            load_chunk<DT>(row, p.V, ch, lane, v);
            const float tot = fold_chunk<DT, true, true>(acc, v, ch, c);
            if (lane == 0) part[ch] = make_float2(acc.ref, tot);
        }
        const float Sw = warp_sum_f(acc.S), Tw = warp_sum_f(acc.T);
        if (lane == 0) {
            WarpRec r;
            r.ref = acc.ref; r.k = acc.k; r.S = Sw; r.T = Tw; r.c1 = acc.c1; r.c2 = acc.c2; r.best = acc.best; r.pad = 0;
            wrec[warp] = r;
        }
        __syncthreads();

        float ref = neg_inf(), Sg = 0.f, Tg = 0.f;
        if (tid == 0) {
            // common reference = the largest of the warps' references; sums rescaled to it in double
            float kref = 0.f;
            bool any_nan = false;
            for (int w = 0; w < kWarps; ++w) {
                if (wrec[w].ref != wrec[w].ref) any_nan = true;
                if (wrec[w].ref > ref) { ref = wrec[w].ref; kref = wrec[w].k; }
            }
            double Sd = 0.0, Td = 0.0;
            for (int w = 0; w < kWarps; ++w) {
                if (wrec[w].ref == neg_inf()) continue;
                const double dd = (double)kref - (double)wrec[w].k;       // <= 0
                const double f = exp2(dd);
                Sd += f * (double)wrec[w].S;
                Td += f * ((double)wrec[w].T + dd * (double)wrec[w].S);
            }
            Sg = (float)Sd; Tg = (float)Td;
            if (any_nan) { Sg = __int_as_float(0x7fc00000); }
            // two largest chunk maxima of the segment (with multiplicity); lowest chunk holding the largest
            float C1 = neg_inf(), C2 = neg_inf();
            int best = -1;
            for (int w = 0; w < kWarps; ++w) {
                const float a1 = wrec[w].c1, a2 = wrec[w].c2;
                if (wrec[w].best < 0) continue;
                if (a1 > C1) { C2 = C1; C1 = a1; best = wrec[w].best; }
                else if (a1 == C1) { C2 = C1; best = min(best, wrec[w].best); }
                else if (a1 > C2) { C2 = a1; }
                if (a2 > C2) C2 = a2;          // a2 <= a1 <= C1 here
            }
            sh_C1 = C1; sh_C2 = C2; sh_best = best;
            sh_cnt = 0; sh_first = 0x7fffffff; sh_below = (int)0x80000000;
        }
        __syncthreads();

        // Second largest element and argmax: only the chunk holding the maximum needs a second look.
        const int best = sh_best;
        const float C1 = sh_C1;
        if (best >= 0) {
            int cnt = 0, first = 0x7fffffff;
            float below = neg_inf();
            for (int e = tid; e < CH; e += kThreads) {
                const int idx = best * CH + e;
                if (idx < p.V) {
                    const float z = load_elem<DT>(row, idx);
                    if (z == C1) { cnt += 1; first = min(first, idx); }
                    else if (z < C1) below = fmaxf(below, z);
                }
            }
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            first = __reduce_min_sync(0xffffffffu, first);
            below = warp_max_f(below);
            if (lane == 0) {
                int bi = __float_as_int(below);
                bi ^= (bi >> 31) & 0x7fffffff;
                atomicAdd(&sh_cnt, cnt);
                atomicMin(&sh_first, first);
                atomicMax(&sh_below, bi);
            }
        }
        __syncthreads();
        if (tid == 0) {
            SegRec r;
            float m2 = sh_C2;
            int am = -1;
            if (best >= 0) {
                int bi = sh_below;
                bi ^= (bi >> 31) & 0x7fffffff;
                const float within = (sh_cnt >= 2) ? C1 : __int_as_float(bi);
                m2 = fmaxf(m2, within);
                am = (sh_first == 0x7fffffff) ? -1 : sh_first;
            }
            r.ref = ref; r.S = Sg; r.T = Tg; r.m2 = m2; r.argmax = am; r.pad0 = r.pad1 = r.pad2 = 0;
            sc.seg[(size_t)s * p.nseg + g] = r;
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

__device__ __forceinline__ RowComb combine_row(const Params& p, const Scratch& sc, int s, float c, int lane) {
    RowComb rc;
    SegRec r;
    r.ref = neg_inf(); r.S = 0.f; r.T = 0.f; r.m2 = neg_inf(); r.argmax = -1;
    if (lane < p.nseg) r = sc.seg[(size_t)s * p.nseg + lane];
    const bool has_nan = __any_sync(0xffffffffu, (r.S != r.S) || (r.T != r.T) || (r.ref != r.ref));
    const float m = warp_max_f(r.ref);
    const unsigned tie = __ballot_sync(0xffffffffu, lane < p.nseg && r.ref == m);
    const int win = tie ? __ffs(tie) - 1 : 0;
    const float other = warp_max_f((lane == win || lane >= p.nseg) ? neg_inf() : r.ref);
    const float m2all = warp_max_f(r.m2);
    rc.m = m;
    rc.m2 = (__popc(tie) >= 2) ? m : fmaxf(other, m2all);
    rc.argmax = __shfl_sync(0xffffffffu, r.argmax, win);
    rc.mc = (double)m * (double)c;
    double Tg = 0.0;
    if (lane < p.nseg && r.ref > neg_inf() && r.ref < CUDART_INF_F) {
        const double d = (double)__fmul_rn(-r.ref, c) + rc.mc;           // >= 0 up to rounding
        Tg = exp2(-d) * ((double)r.T - d * (double)r.S);
    }
    rc.T2 = warp_sum_d(Tg);
    rc.tot = cdf_totals(sc.cdf + (size_t)s * p.NC, p.NC, c, rc.mc, true, lane);
    rc.W = rc.tot.W;
    rc.valid = !has_nan && (m > neg_inf()) && (m < CUDART_INF_F) && (rc.W > 0.0) && (rc.W < CUDART_INF);
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
               int parity, uint32_t round, float c, int32_t* __restrict__ out_token, long long tok_stride,
               uint8_t* __restrict__ out_continue)
{
    constexpr int CH = chunk_elems<DT>();
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

    const RowComb rc = combine_row(p, sc, s, c, lane);
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
    const char* row = reinterpret_cast<const char*>(logits) + (size_t)s * row_stride * Elem<DT>::BYTES;
    const uint4 w = rng_words(p, seq, round, (uint32_t)pos, RNG_DRAFT, 0, 0);
    const double u = u24_to_double(w.x);
    double rem;
    const int chunk = cdf_locate(sc.cdf + (size_t)s * p.NC, p.NC, c, rc.mc, true, lane, rc.tot, u * rc.W, rem);
    const double inv_T = (double)p.inv_Tq, m_s = f.m_s;
    const int tok = pick_in_chunk<CH>(chunk, p.V, rem, lane,
                                      [&](int idx) { return exp((double)load_elem<DT>(row, idx) * inv_T - m_s); });

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
__global__ void __launch_bounds__(128)
k_rows_features(Params p, Scratch sc, int n_rows, float c, float inv_T, float* __restrict__ out)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int s = blockIdx.x * 4 + warp;
    if (s >= n_rows) return;
    const RowComb rc = combine_row(p, sc, s, c, lane);
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
    constexpr int CH = chunk_elems<DT>();
    constexpr int ESZ = Elem<DT>::BYTES;
    extern __shared__ float2 sm_part[];
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
                    const double iTp = (double)p.inv_Tp, iTq = (double)p.inv_Tq;
                    tok = pick_in_chunk<CH>(chunk, p.V, rem * exp2(-dq), lane, [&](int idx) {
                        const double r = exp((double)load_elem<DT>(prow, idx) * iTp - lse_p) -
                                         exp((double)load_elem<DT>(qrow, idx) * iTq - lse_q);
                        return r > 0.0 ? r : 0.0;
                    });
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
                    const double iTp = (double)p.inv_Tp, m_s = (double)m_p * iTp;
                    const int tok = pick_in_chunk<CH>(chunk, p.V, rem, lane, [&](int idx) {
                        return exp((double)load_elem<DT>(prow, idx) * iTp - m_s);
                    });
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
