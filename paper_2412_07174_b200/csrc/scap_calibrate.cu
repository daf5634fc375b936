// Offline calibration (Section 3; Eq. 2): per-channel mode by histogram arg-max, then the pooled
// quantile of |x - m| by a three-pass radix select on the binary32 bit pattern (non-negative floats
// order like their unsigned bit patterns).  All value arithmetic uses the *_rn intrinsics so that no
// multiply-add is contracted and results are bit-reproducible.
#include <math.h>

#include "scap_common.cuh"

namespace scap {

constexpr int CW = 32;             // channels per CTA strip: 4 threads x 8 channels (16 B) per row
constexpr int CAL_THREADS = 512;   // 128 rows per sweep
constexpr int CAL_ROWS = CAL_THREADS / 4;
constexpr int RADIX_BINS = 2048;   // 11 bits per pass; passes take bits 30..20, 19..9, 8..0

struct SelState {
    uint32_t prefix[2];  // key bits decided so far for order statistics j and j+1
    uint32_t rank[2];    // rank of each within the keys that share its prefix
};

template <bool BF16>
__device__ __forceinline__ void widen8(const uint4 &v, float (&f)[8]) {
    widen2<BF16>(v.x, f[0], f[1]);
    widen2<BF16>(v.y, f[2], f[3]);
    widen2<BF16>(v.z, f[4], f[5]);
    widen2<BF16>(v.w, f[6], f[7]);
}

// Rows t0, t0 + CAL_ROWS, ... (CAL_U of them) of this thread's 8 channels, all loads in flight together; rows at or
// beyond T are skipped (their slots keep zeros and `valid` says how many are real).
constexpr int CAL_U = 16;  // with 128 rows per sweep: 2048 rows of a strip live in registers at once
__device__ __forceinline__ int load_rows(const uint16_t *xp, int K, int T, int t0, uint4 (&v)[CAL_U]) {
    const uint64_t pol = l2_policy_keep();  // the radix passes read the tensor again: it fits in L2, ask for it to stay
    int valid = 0;
#pragma unroll
    for (int u = 0; u < CAL_U; ++u) {
        const int t = t0 + u * CAL_ROWS;
        v[u] = make_uint4(0, 0, 0, 0);
        if (t < T) {
            v[u] = ld_keep16(xp + (size_t)t * K, pol);
            valid = u + 1;
        }
    }
    return valid;
}

// Rotates the 8 channels of a 16-byte row piece by r places: channel i of the result is channel (i + r) mod 8 of v.
// Branch-free (r differs between the lanes of a warp).
__device__ __forceinline__ uint4 rotate_channels(const uint4 &v, int r) {
    uint32_t w0 = v.x, w1 = v.y, w2 = v.z, w3 = v.w;
    {
        const bool on = (r & 1) != 0;  // one channel = 16 bits
        const uint32_t t0 = __funnelshift_r(w0, w1, 16), t1 = __funnelshift_r(w1, w2, 16);
        const uint32_t t2 = __funnelshift_r(w2, w3, 16), t3 = __funnelshift_r(w3, w0, 16);
        w0 = on ? t0 : w0; w1 = on ? t1 : w1; w2 = on ? t2 : w2; w3 = on ? t3 : w3;
    }
    {
        const bool on = (r & 2) != 0;  // two channels = one word
        const uint32_t t0 = w1, t1 = w2, t2 = w3, t3 = w0;
        w0 = on ? t0 : w0; w1 = on ? t1 : w1; w2 = on ? t2 : w2; w3 = on ? t3 : w3;
    }
    {
        const bool on = (r & 4) != 0;  // four channels = two words
        const uint32_t t0 = w2, t1 = w3, t2 = w0, t3 = w1;
        w0 = on ? t0 : w0; w1 = on ? t1 : w1; w2 = on ? t2 : w2; w3 = on ? t3 : w3;
    }
    return make_uint4(w0, w1, w2, w3);
}

// One CTA per strip of CWT channels (32: 512 threads, one CTA per SM; 16: 256 threads, two CTAs per SM, finer
// strips that spread better over the SMs): min/max, histogram, arg-max -> m; then the first radix histogram
// (bits 30..20 of |x - m|) of the strip is added to hist_a.
//
// Histogram layout: the two 16-bit counters of bins 2h and 2h+1 of channel c share word h * CW + c, so the bank of
// a counter is its channel (CWT = 32; with 16 channels two bin pairs share a row of banks).  A warp holds 8 rows x 4
// pieces (16 rows x 2 pieces) of 8 channels; each lane rotates its 8 channels by its row number, so that in every
// step of the unrolled loop the lanes of a warp update CWT different channels: with 32 channels no two lanes ever
// meet in a bank, whatever the bins; with 16 channels two lanes can.
template <bool BF16, int CWT>
__global__ void __launch_bounds__(CWT * 16, CWT == 16 ? 2 : 1) mode_kernel(const uint16_t *__restrict__ x, int T, int K, int nbins,
                                                           float *__restrict__ m_out, uint32_t *__restrict__ hist_a,
                                                           int want_hist, const float *__restrict__ m_given) {
    griddep_wait();               // m_given and the cleared counters come from earlier work on the stream
    griddep_launch_dependents();  // the next pass may become resident early; it waits for this grid itself
    constexpr int QN = CWT / 8;        // 16-byte pieces per row of the strip
    constexpr int NTH = QN * CAL_ROWS;  // threads: 128 rows per sweep
    constexpr int NW = NTH / 32;
    extern __shared__ __align__(16) uint32_t smem[];
    __shared__ float s_lo[CWT], s_hi[CWT], s_m[CWT];
    __shared__ float s_wlo[NW][CWT], s_whi[NW][CWT];  // per-warp partial min / max, later partial arg-max (count, bin)
    const int tid = threadIdx.x, q = tid % QN, rl = tid / QN;
    const int lane = tid & 31, warp = tid >> 5, r = (lane / QN) & 7;
    const int k0 = blockIdx.x * CWT;
    const int kc = k0 + q * 8;
    const bool ok = kc < K;  // K is a multiple of 8
    const uint16_t *xp = x + kc;
    // Up to CAL_ROWS * CAL_U = 2048 rows: the strip is read once, all loads in flight together, and the three
    // passes below run from registers; longer inputs are re-read per pass (from L2 when they fit).
    const bool resident = T <= CAL_ROWS * CAL_U;
    uint4 v[CAL_U];
    int nv = 0;
    if (resident && ok) nv = load_rows(xp, K, T, rl, v);

    if (m_given) {  // the mode was estimated by another kernel: only the radix histogram below is wanted
        if (tid < CWT) s_m[tid] = k0 + tid < K ? __ldcg(m_given + k0 + tid) : 0.0f;
        __syncthreads();
    } else if (nbins > 0) {
        // ---- pass 1: per-channel min / max (thread -> 8 rows of the warp by shuffles -> warps through shared memory)
        float lo[8], hi[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { lo[j] = INFINITY; hi[j] = -INFINITY; }
        if (ok)
            for (int t0 = rl; t0 < T; t0 += CAL_ROWS * CAL_U) {
                if (!resident) nv = load_rows(xp, K, T, t0, v);
#pragma unroll
                for (int u = 0; u < CAL_U; ++u) {
                    if (u < nv) {
                        float f[8];
                        widen8<BF16>(v[u], f);
#pragma unroll
                        for (int j = 0; j < 8; ++j) { lo[j] = fminf(lo[j], f[j]); hi[j] = fmaxf(hi[j], f[j]); }
                    }
                }
            }
#pragma unroll
        for (int o = QN; o < 32; o <<= 1)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                lo[j] = fminf(lo[j], __shfl_xor_sync(0xffffffffu, lo[j], o));
                hi[j] = fmaxf(hi[j], __shfl_xor_sync(0xffffffffu, hi[j], o));
            }
        if (lane < QN) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                s_wlo[warp][q * 8 + j] = lo[j];
                s_whi[warp][q * 8 + j] = hi[j];
            }
        }
        __syncthreads();
        if (tid < CWT) {
            float l = INFINITY, h = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) { l = fminf(l, s_wlo[w][tid]); h = fmaxf(h, s_whi[w][tid]); }
            s_lo[tid] = l;
            s_hi[tid] = h;
        }
        // ---- pass 2: histogram; two 16-bit counters per word (a count never exceeds T <= 65535)
        const int HW = (nbins + 1) / 2;
        for (int i = tid; i < CWT * HW; i += NTH) smem[i] = 0;
        __syncthreads();
        // this lane's channels in rotated order: slot i holds channel q * 8 + (i + r) mod 8
        float scale[8];
        int cidx[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            cidx[i] = q * 8 + ((i + r) & 7);
            lo[i] = s_lo[cidx[i]];
            hi[i] = s_hi[cidx[i]];
            scale[i] = hi[i] != lo[i] ? __fdiv_rn((float)nbins, __fsub_rn(hi[i], lo[i])) : 0.0f;
        }
        if (ok)
            for (int t0 = rl; t0 < T; t0 += CAL_ROWS * CAL_U) {
                if (!resident) nv = load_rows(xp, K, T, t0, v);
#pragma unroll
                for (int u = 0; u < CAL_U; ++u) {
                    if (u < nv) {
                        float f[8];
                        widen8<BF16>(rotate_channels(v[u], r), f);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            // floor of the non-negative product without a conversion instruction: adding 2^23
                            // rounding down leaves floor(v) in the mantissa (exact for 0 <= v < 2^23).  A constant
                            // channel has scale 0 and counts into bin 0; its mode is set from lo below.
                            const float vb = __fmul_rn(__fsub_rn(f[i], lo[i]), scale[i]);
                            int b = __float_as_int(__fadd_rd(vb, 8388608.0f)) & 0x7fffff;
                            b = min(b, nbins - 1);
                            atomicAdd(&smem[(b >> 1) * CWT + cidx[i]], 1u << ((b & 1) * 16));
                        }
                    }
                }
            }
        __syncthreads();
        // ---- arg-max: lowest bin with the largest count.  A lane scans bin pairs of channel lane mod CWT in ascending
        // order (strict >: the first maximum stays); with 16 channels the two half-warps take alternate pairs and
        // are merged by (count, then lower bin).  Thread c then combines the warps in ascending order.
        {
            constexpr int LS = 32 / CWT;  // lanes per channel in a warp
            const int per = (HW + NW - 1) / NW;
            const int sub = lane / CWT, ch = lane % CWT;
            uint32_t best_cnt = 0;
            int best_i = 0;
            const int h_end = min(HW, (warp + 1) * per);
            for (int h0 = warp * per + sub; h0 < h_end; h0 += 8 * LS) {
                uint32_t wv[8];  // eight independent loads, then the ordered compares
#pragma unroll
                for (int e = 0; e < 8; ++e) wv[e] = h0 + e * LS < h_end ? smem[(h0 + e * LS) * CWT + ch] : 0u;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const uint32_t c0 = wv[e] & 0xffffu, c1 = wv[e] >> 16;  // bin 2h + 1 beyond nbins was never counted
                    if (c0 > best_cnt) { best_cnt = c0; best_i = 2 * (h0 + e * LS); }
                    if (c1 > best_cnt) { best_cnt = c1; best_i = 2 * (h0 + e * LS) + 1; }
                }
            }
            if constexpr (LS == 2) {
                const uint32_t oc = __shfl_xor_sync(0xffffffffu, best_cnt, 16);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, 16);
                if (oc > best_cnt || (oc == best_cnt && oi < best_i)) { best_cnt = oc; best_i = oi; }
            }
            if (sub == 0) {
                s_wlo[warp][ch] = __uint_as_float(best_cnt);
                s_whi[warp][ch] = __int_as_float(best_i);
            }
        }
        __syncthreads();
        if (tid < CWT) {
            uint32_t best_cnt = 0;
            int best_i = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const uint32_t c = __float_as_uint(s_wlo[w][tid]);
                if (c > best_cnt) { best_cnt = c; best_i = __float_as_int(s_whi[w][tid]); }
            }
            const float l = s_lo[tid], h = s_hi[tid];
            float mv = l;
            if (h != l) {
                const float w = __fmul_rn(__fsub_rn(h, l), __fdiv_rn(1.0f, (float)nbins));
                mv = __fadd_rn(l, __fmul_rn(__fadd_rn((float)best_i, 0.5f), w));
            }
            s_m[tid] = mv;
            if (k0 + tid < K) m_out[k0 + tid] = mv;
        }
        __syncthreads();
    } else {
        if (tid < CWT) {
            s_m[tid] = 0.0f;
            if (k0 + tid < K) m_out[k0 + tid] = 0.0f;
        }
        __syncthreads();
    }
    if (!want_hist) return;
    // ---- pass 3: first radix histogram of the importance |x - m|.  The keys crowd into a few dozen buckets (the
    // top 11 bits are the exponent and three mantissa bits), so groups of four neighbouring lanes count into four
    // copies of the histogram, each shifted by 8 banks against the previous one.
    for (int i = tid; i < 4 * RADIX_BINS; i += NTH) smem[i] = 0;
    float mk[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) mk[j] = s_m[q * 8 + j];
    __syncthreads();
    const int cp = lane & 3;  // copy of this lane
    uint32_t *hq = smem + cp * RADIX_BINS;
    if (ok)
        for (int t0 = rl; t0 < T; t0 += CAL_ROWS * CAL_U) {
            if (!resident) nv = load_rows(xp, K, T, t0, v);
#pragma unroll
            for (int u = 0; u < CAL_U; ++u) {
                if (u < nv) {
                    float f[8];
                    widen8<BF16>(v[u], f);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t key = __float_as_uint(__fsub_rn(f[j], mk[j])) & 0x7fffffffu;
                        atomicAdd(&hq[((key >> 20) + 8 * cp) & (RADIX_BINS - 1)], 1u);
                    }
                }
            }
        }
    __syncthreads();
    for (int i = tid; i < RADIX_BINS; i += NTH) {
        uint32_t c = 0;
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) c += smem[qq * RADIX_BINS + ((i + 8 * qq) & (RADIX_BINS - 1))];
        if (c) atomicAdd(&hist_a[i], c);
    }
}

// Block-wide bucket search (256 threads): for the order statistics w = 0, 1, finds in the nb counters h[w] (nb a
// multiple of 256, at most 2048) the bucket that holds rank[w] (0-based among the counted keys) and rebases the rank
// to that bucket.  Every thread returns both results.  Thread t adds its nb / 256 consecutive counters, the block
// scans the 256 sums, and the one thread whose stretch contains the rank walks its own counters.
struct SelPick {
    uint32_t bucket[2], rank[2];
};
__device__ __forceinline__ SelPick block_select(const uint32_t *const (&h)[2], int nb, const uint32_t (&rank)[2]) {
    __shared__ uint32_t s_wsum[2][8];
    __shared__ uint32_t s_pick[2][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = nb >> 8;  // 1 .. 8
    uint32_t cnt[2][8], incl[2];
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        uint32_t sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            cnt[w][i] = i < per ? __ldcg(h[w] + tid * per + i) : 0u;
            sum += cnt[w][i];
        }
        uint32_t v = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += t;
        }
        incl[w] = v;
        if (lane == 31) s_wsum[w][warp] = v;
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < 2; ++w) {
        uint32_t before = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) before += q < warp ? s_wsum[w][q] : 0u;
        uint32_t sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) sum += cnt[w][i];
        uint32_t lo = before + incl[w] - sum;  // keys in the buckets before this thread's stretch
        if (rank[w] >= lo && rank[w] < lo + sum) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (rank[w] >= lo && rank[w] < lo + cnt[w][i]) {
                    s_pick[w][0] = (uint32_t)(tid * per + i);
                    s_pick[w][1] = rank[w] - lo;
                }
                lo += cnt[w][i];
            }
        }
    }
    __syncthreads();
    SelPick r;
    r.bucket[0] = s_pick[0][0]; r.rank[0] = s_pick[0][1];
    r.bucket[1] = s_pick[1][0]; r.rank[1] = s_pick[1][1];
    return r;
}

// Radix passes after the first: histogram of the next `width` key bits over the elements whose higher bits equal
// the prefix of order statistic j (hist[0]) or j+1 (hist[1]).
// Each CTA first extends the two prefixes itself from the previous pass's counters (block_select: every CTA gets
// the same answer, so no separate one-CTA kernel sits between two passes); CTA (0, 0) records them in st_out.
// A CTA owns a block of 256 channels (32 lanes x 8 channels: a warp reads 512 contiguous bytes of a row) and the
// rows blockIdx.y * 8 + ty, stepping by 8 * gridDim.y; the modes of a thread's 8 channels stay in registers.
// With t = key - (prefix << (shift + width)) as unsigned, the higher bits match iff t < 2^(shift + width), and
// t >> shift is then the bucket.  The two order statistics are neighbours and nearly always share their prefix:
// then one histogram is counted and added to both outputs.
constexpr int RP_U = 8;  // 16-byte loads in flight per thread
template <bool BF16>
__global__ void __launch_bounds__(256) radix_pass_kernel(const uint16_t *__restrict__ x, const float *__restrict__ m, int T,
                                                         int K, const uint32_t *__restrict__ prev_hist, int prev_two,
                                                         int prev_width, const SelState *__restrict__ st_in, uint32_t j,
                                                         uint32_t j1, SelState *__restrict__ st_out, int shift, int width,
                                                         uint32_t *__restrict__ hist) {
    __shared__ uint32_t s_h[2][RADIX_BINS];
    for (int i = threadIdx.x; i < 2 * RADIX_BINS; i += blockDim.x) (&s_h[0][0])[i] = 0;
    griddep_wait();               // the previous pass's counters are complete
    griddep_launch_dependents();
    const int sh = shift + width;
    // previous pass: one shared histogram (the first pass) or one per order statistic
    const uint32_t *const ph[2] = {prev_hist, prev_two ? prev_hist + RADIX_BINS : prev_hist};
    const uint32_t rk[2] = {st_in ? st_in->rank[0] : j, st_in ? st_in->rank[1] : j1};
    const SelPick pick = block_select(ph, RADIX_BINS, rk);
    const uint32_t p0 = ((st_in ? st_in->prefix[0] : 0u) << prev_width) | pick.bucket[0];
    const uint32_t p1 = ((st_in ? st_in->prefix[1] : 0u) << prev_width) | pick.bucket[1];
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        st_out->prefix[0] = p0; st_out->prefix[1] = p1;
        st_out->rank[0] = pick.rank[0]; st_out->rank[1] = pick.rank[1];
    }
    const uint32_t base0 = p0 << sh, base1 = p1 << sh, span = 1u << sh;
    const bool same = p0 == p1;
    const int kc = (blockIdx.x * 32 + (threadIdx.x & 31)) * 8;
    const int ty = threadIdx.x >> 5;
    float mk[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) mk[jj] = 0.0f;
    if (kc < K) {
        const float4 ma = __ldg(reinterpret_cast<const float4 *>(m + kc)), mb = __ldg(reinterpret_cast<const float4 *>(m + kc + 4));
        mk[0] = ma.x; mk[1] = ma.y; mk[2] = ma.z; mk[3] = ma.w;
        mk[4] = mb.x; mk[5] = mb.y; mk[6] = mb.z; mk[7] = mb.w;
    }
    __syncthreads();
    if (kc < K) {
        const int step = 8 * gridDim.y;
        const uint16_t *xp = x + kc;
        const uint64_t pol = l2_policy_keep();
        for (int t0 = blockIdx.y * 8 + ty; t0 < T; t0 += step * RP_U) {
            uint4 v[RP_U];
#pragma unroll
            for (int u = 0; u < RP_U; ++u) {
                const int t = t0 + step * u;
                v[u] = make_uint4(0, 0, 0, 0);
                if (t < T) v[u] = ld_keep16(xp + (size_t)t * K, pol);
            }
#pragma unroll
            for (int u = 0; u < RP_U; ++u) {
                if (t0 + step * u < T) {
                    float f[8];
                    widen8<BF16>(v[u], f);
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const uint32_t key = __float_as_uint(__fsub_rn(f[jj], mk[jj])) & 0x7fffffffu;
                        const uint32_t d0 = key - base0;
                        if (d0 < span) atomicAdd(&s_h[0][d0 >> shift], 1u);
                        if (!same) {
                            const uint32_t d1 = key - base1;
                            if (d1 < span) atomicAdd(&s_h[1][d1 >> shift], 1u);
                        }
                    }
                }
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < RADIX_BINS; i += blockDim.x) {
        const uint32_t c0 = s_h[0][i], c1 = same ? c0 : s_h[1][i];
        if (c0) atomicAdd(&hist[i], c0);
        if (c1) atomicAdd(&hist[RADIX_BINS + i], c1);
    }
}

// One CTA of 256 threads, after the last pass: finds the last `width` key bits of both order statistics in
// hist[0] / hist[1] (nb counters each) and interpolates
// tau = v_j + frac * (v_j1 - v_j) in binary64, each operation rounded once, then rounded to binary32.
__global__ void __launch_bounds__(256) select_kernel(const uint32_t *__restrict__ hist, int nb, int width,
                                                     const SelState *__restrict__ st_in, double frac,
                                                     float *__restrict__ tau_out) {
    griddep_wait();
    const uint32_t *const ph[2] = {hist, hist + RADIX_BINS};
    const uint32_t rk[2] = {st_in->rank[0], st_in->rank[1]};
    const SelPick pick = block_select(ph, nb, rk);
    if (threadIdx.x == 0) {
        const double vj = (double)__uint_as_float((st_in->prefix[0] << width) | pick.bucket[0]);
        const double vj1 = (double)__uint_as_float((st_in->prefix[1] << width) | pick.bucket[1]);
        const double t64 = __dadd_rn(vj, __dmul_rn(frac, __dsub_rn(vj1, vj)));
        *tau_out = (float)t64;
    }
}

__global__ void set_float_kernel(float *p, float v) { *p = v; }


// ---------------------------------------------------------------------------------------------------------
// Other estimators of the mode (Section 3, "Determination of mode value": mean, median) and the paper's scalar
// eta (one value for the whole FC input instead of one per channel).
// ---------------------------------------------------------------------------------------------------------

template <bool BF16>
__device__ __forceinline__ float widen16(uint16_t u) {
    if constexpr (BF16) return __uint_as_float((uint32_t)u << 16);
    else return __half2float(__ushort_as_half(u));
}

// Monotone 16-bit key of a 16-bit float pattern (ascending values <-> ascending keys) and its inverse.
__device__ __forceinline__ uint32_t key16(uint16_t u) { return (u & 0x8000u) ? (uint32_t)(uint16_t)~u : (uint32_t)(u | 0x8000u); }
__device__ __forceinline__ uint16_t unkey16(uint32_t k) { return (k & 0x8000u) ? (uint16_t)(k & 0x7fffu) : (uint16_t)~k; }

// Mean: a CTA owns 32 channels.  All threads stage tiles of 64 rows in shared memory (16-byte loads, the next tile
// in flight while the current one is consumed); thread c < 32 adds column c of each tile in row order in binary64
// (the definition fixes the order).  Writes the rounded mean and, for the scalar form, the unrounded column sum.
template <bool BF16>
__global__ void __launch_bounds__(256) mean_kernel(const uint16_t *__restrict__ x, int T, int K, float *__restrict__ m_out,
                                                   double *__restrict__ col_sum) {
    __shared__ __align__(16) uint16_t s_t[2][64][32];
    const int tid = threadIdx.x, row = tid >> 2, q = tid & 3;
    const int k0 = blockIdx.x * 32, kc = k0 + q * 8;
    const bool ok = kc < K;  // K is a multiple of 8
    const uint16_t *xp = x + kc;
    const int ntiles = (T + 63) / 64;
    auto fetch = [&](int i) {
        const int t = i * 64 + row;
        return (ok && t < T) ? __ldg(reinterpret_cast<const uint4 *>(xp + (size_t)t * K)) : make_uint4(0, 0, 0, 0);
    };
    uint4 r = fetch(0);
    *reinterpret_cast<uint4 *>(&s_t[0][row][q * 8]) = r;
    __syncthreads();
    double acc = 0.0;
    for (int i = 0; i < ntiles; ++i) {
        if (i + 1 < ntiles) r = fetch(i + 1);
        if (tid < 32) {
            const int n = min(64, T - i * 64);
#pragma unroll 8
            for (int j = 0; j < n; ++j) acc = __dadd_rn(acc, (double)widen16<BF16>(s_t[i & 1][j][tid]));
        }
        if (i + 1 < ntiles) *reinterpret_cast<uint4 *>(&s_t[(i + 1) & 1][row][q * 8]) = r;
        __syncthreads();
    }
    if (tid < 32 && k0 + tid < K) {
        if (m_out) m_out[k0 + tid] = __fadd_rn((float)__ddiv_rn(acc, (double)T), 0.0f);
        if (col_sum) col_sum[k0 + tid] = acc;
    }
}

// One CTA: the sums are staged in shared memory 2048 at a time (all threads), thread 0 adds them in order.
__global__ void __launch_bounds__(256) eta_mean_kernel(const double *__restrict__ col_sum, int T, int K, float *__restrict__ eta) {
    __shared__ double s_v[2048];
    double total = 0.0;
    for (int k0 = 0; k0 < K; k0 += 2048) {
        const int n = min(2048, K - k0);
        for (int i = threadIdx.x; i < n; i += blockDim.x) s_v[i] = __ldcg(col_sum + k0 + i);
        __syncthreads();
        if (threadIdx.x == 0)
            for (int i = 0; i < n; ++i) total = __dadd_rn(total, s_v[i]);
        __syncthreads();
    }
    if (threadIdx.x == 0) *eta = __fadd_rn((float)__ddiv_rn(total, __dmul_rn((double)T, (double)K)), 0.0f);
}

__global__ void broadcast_kernel(float *__restrict__ m_out, int K, const float *__restrict__ eta) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < K) m_out[k] = __ldcg(eta);
}

// Finds, in a 256-bin histogram h, the bin that holds rank r (0-based) and the rank inside that bin.  One warp.
__device__ __forceinline__ void find_rank256(const uint32_t *h, uint32_t r, int lane, uint32_t &bin, uint32_t &inner) {
    uint32_t c[8], tot = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = h[lane * 8 + i]; tot += c[i]; }
    uint32_t incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    uint32_t excl = incl - tot;
    const unsigned hit = __ballot_sync(0xffffffffu, r >= excl && r < incl);
    const int src = hit ? __ffs(hit) - 1 : 31;
    uint32_t b = 0, in = 0;
    if (lane == src) {
        uint32_t run = excl;
        b = 7; in = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (r >= run && r < run + c[i]) { b = (uint32_t)i; in = r - run; }
            run += c[i];
        }
        b += (uint32_t)lane * 8;
    }
    bin = __shfl_sync(0xffffffffu, b, src);
    inner = __shfl_sync(0xffffffffu, in, src);
}

// Median per channel: two 8-bit radix passes over the 16-bit keys of a strip of CW channels, from registers.
// Shared memory: hi[CW][256] | lo[2][CW][256] counters | per-channel bucket state.
template <bool BF16>
__global__ void __launch_bounds__(CAL_THREADS) median_kernel(const uint16_t *__restrict__ x, int T, int K, float *__restrict__ m_out) {
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t *s_hi = smem, *s_lo = smem + CW * 256;
    __shared__ uint32_t s_bucket[2][CW], s_inner[2][CW];
    const int tid = threadIdx.x, q = tid & 3, rl = tid >> 2, lane = tid & 31, warp = tid >> 5;
    const int k0 = blockIdx.x * CW, kc = k0 + q * 8;
    const bool ok = kc < K;
    const uint16_t *xp = x + kc;
    const bool resident = T <= CAL_ROWS * CAL_U;
    uint4 v[CAL_U];
    int nv = 0;
    if (resident && ok) nv = load_rows(xp, K, T, rl, v);
    for (int i = tid; i < 3 * CW * 256; i += CAL_THREADS) smem[i] = 0;
    __syncthreads();
    // pass A: high byte
    if (ok)
        for (int t0 = rl; t0 < T; t0 += CAL_ROWS * CAL_U) {
            if (!resident) nv = load_rows(xp, K, T, t0, v);
#pragma unroll
            for (int u = 0; u < CAL_U; ++u) {
                if (u < nv) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t key = key16((uint16_t)(w[j >> 1] >> ((j & 1) * 16)));
                        atomicAdd(&s_hi[(q * 8 + j) * 256 + (key >> 8)], 1u);
                    }
                }
            }
        }
    __syncthreads();
    const uint32_t r0 = (uint32_t)(T - 1) / 2, r1 = (uint32_t)T / 2;
    for (int c = warp * (CW / (CAL_THREADS / 32)); c < (warp + 1) * (CW / (CAL_THREADS / 32)); ++c) {
        uint32_t b, in;
        find_rank256(s_hi + c * 256, r0, lane, b, in);
        if (lane == 0) { s_bucket[0][c] = b; s_inner[0][c] = in; }
        find_rank256(s_hi + c * 256, r1, lane, b, in);
        if (lane == 0) { s_bucket[1][c] = b; s_inner[1][c] = in; }
    }
    __syncthreads();
    // pass B: low byte inside the two buckets
    if (ok)
        for (int t0 = rl; t0 < T; t0 += CAL_ROWS * CAL_U) {
            if (!resident) nv = load_rows(xp, K, T, t0, v);
#pragma unroll
            for (int u = 0; u < CAL_U; ++u) {
                if (u < nv) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int c = q * 8 + j;
                        const uint32_t key = key16((uint16_t)(w[j >> 1] >> ((j & 1) * 16)));
                        if ((key >> 8) == s_bucket[0][c]) atomicAdd(&s_lo[c * 256 + (key & 255u)], 1u);
                        if ((key >> 8) == s_bucket[1][c]) atomicAdd(&s_lo[(CW + c) * 256 + (key & 255u)], 1u);
                    }
                }
            }
        }
    __syncthreads();
    for (int c = warp * (CW / (CAL_THREADS / 32)); c < (warp + 1) * (CW / (CAL_THREADS / 32)); ++c) {
        uint32_t b0, b1, in;
        find_rank256(s_lo + c * 256, s_inner[0][c], lane, b0, in);
        find_rank256(s_lo + (CW + c) * 256, s_inner[1][c], lane, b1, in);
        if (lane == 0 && k0 + c < K) {
            const double lo = (double)widen16<BF16>(unkey16((s_bucket[0][c] << 8) | b0));
            const double hi = (double)widen16<BF16>(unkey16((s_bucket[1][c] << 8) | b1));
            m_out[k0 + c] = __fadd_rn((float)__ddiv_rn(__dadd_rn(lo, hi), 2.0), 0.0f);
        }
    }
}

// KDE peak per channel (Section 3 names the KDE next to the mean and the median): Gaussian kernel, bandwidth
// h = sigma * T^(-1/5) with the sample standard deviation (divisor T - 1), density on G grid points between the
// channel's minimum and maximum, first point of largest density.  All in binary64.
// One CTA of 256 threads per strip of 8 channels: the strip is staged in shared memory as binary32 (exact for
// 16-bit inputs), warp c computes the statistics of channel c, then for each channel every thread evaluates the
// grid points tid, tid + 256, ... (all T samples each, read as shared-memory broadcasts) and the block keeps the
// best (density, then lower index).
constexpr int KDE_MAX_T = 4096;
template <bool BF16>
__global__ void __launch_bounds__(256) kde_kernel(const uint16_t *__restrict__ x, int T, int K, int G, float *__restrict__ m_out) {
    extern __shared__ __align__(16) float s_x[];  // [8][T]
    __shared__ float s_lo[8], s_hi[8];
    __shared__ double s_h[8];
    __shared__ double s_bd[8];
    __shared__ int s_bi[8];
    griddep_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int k0 = blockIdx.x * 8;  // K is a multiple of 8
    for (int t = tid; t < T; t += 256) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x + (size_t)t * K + k0));
        float f[8];
        widen8<BF16>(v, f);
#pragma unroll
        for (int j = 0; j < 8; ++j) s_x[j * T + t] = f[j];
    }
    __syncthreads();
    {  // statistics of channel `warp`
        const float *xc = s_x + warp * T;
        float lo = INFINITY, hi = -INFINITY;
        double sum = 0.0;
        for (int t = lane; t < T; t += 32) {
            const float v = xc[t];
            lo = fminf(lo, v);
            hi = fmaxf(hi, v);
            sum += (double)v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
            sum += __shfl_xor_sync(0xffffffffu, sum, o);
        }
        const double mu = sum / (double)T;
        double ss = 0.0;
        for (int t = lane; t < T; t += 32) {
            const double d = (double)xc[t] - mu;
            ss += d * d;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) {
            s_lo[warp] = lo;
            s_hi[warp] = hi;
            s_h[warp] = T > 1 ? sqrt(ss / (double)(T - 1)) * pow((double)T, -0.2) : 0.0;
        }
    }
    __syncthreads();
    for (int c = 0; c < 8; ++c) {
        const float lo = s_lo[c], hi = s_hi[c];
        if (hi == lo) {  // constant channel (block-uniform)
            if (tid == 0) m_out[k0 + c] = lo + 0.0f;
            continue;
        }
        const float *xc = s_x + c * T;
        const double inv_h = 1.0 / s_h[c];
        const double step = ((double)hi - (double)lo) / (double)(G - 1);
        double best = -1.0;
        int best_i = 0x7fffffff;
        for (int i = tid; i < G; i += 256) {
            const double g = (double)lo + (double)i * step;
            double d0 = 0.0, d1 = 0.0;
            int t = 0;
            for (; t + 1 < T; t += 2) {  // two independent chains
                const double u0 = (g - (double)xc[t]) * inv_h, u1 = (g - (double)xc[t + 1]) * inv_h;
                d0 += exp(-0.5 * (u0 * u0));
                d1 += exp(-0.5 * (u1 * u1));
            }
            if (t < T) {
                const double u0 = (g - (double)xc[t]) * inv_h;
                d0 += exp(-0.5 * (u0 * u0));
            }
            const double dens = d0 + d1;
            if (dens > best) { best = dens; best_i = i; }  // ascending i per thread: the first maximum stays
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
            if (od > best || (od == best && oi < best_i)) { best = od; best_i = oi; }
        }
        if (lane == 0) { s_bd[warp] = best; s_bi[warp] = best_i; }
        __syncthreads();
        if (tid == 0) {
            double bd = s_bd[0];
            int bi = s_bi[0];
            for (int w = 1; w < 8; ++w)
                if (s_bd[w] > bd || (s_bd[w] == bd && s_bi[w] < bi)) { bd = s_bd[w]; bi = s_bi[w]; }
            m_out[k0 + c] = (float)((double)lo + (double)bi * step) + 0.0f;
        }
        __syncthreads();
    }
}

// Pooled (whole-tensor) statistics for the scalar eta.
struct PoolState {
    uint32_t bucket[2], inner[2];  // median: high-byte bucket and rank inside it, for the two middle ranks
    int lo_key, hi_key;            // histogram mode: ordered-integer images of the minimum and the maximum
    float eta;
};

__device__ __forceinline__ int ordered_int(float f) { const int i = __float_as_int(f); return i >= 0 ? i : i ^ 0x7fffffff; }
__device__ __forceinline__ float from_ordered_int(int i) { return __int_as_float(i >= 0 ? i : i ^ 0x7fffffff); }

// pass 0: histogram of the high key byte; pass 1: of the low byte inside the two buckets found after pass 0.
template <bool BF16>
__global__ void __launch_bounds__(256) pooled_key_hist_kernel(const uint16_t *__restrict__ x, long long M8, int pass,
                                                              const PoolState *__restrict__ st, uint32_t *__restrict__ hist) {
    __shared__ uint32_t s_h[2][256];
    for (int i = threadIdx.x; i < 512; i += blockDim.x) (&s_h[0][0])[i] = 0;
    const uint32_t bk0 = pass ? st->bucket[0] : 0u, bk1 = pass ? st->bucket[1] : 0u;
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < M8; i += stride) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x) + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t key = key16((uint16_t)(w[j >> 1] >> ((j & 1) * 16)));
            if (pass == 0) {
                atomicAdd(&s_h[0][key >> 8], 1u);
            } else {
                if ((key >> 8) == bk0) atomicAdd(&s_h[0][key & 255u], 1u);
                if ((key >> 8) == bk1) atomicAdd(&s_h[1][key & 255u], 1u);
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 512; i += blockDim.x) {
        const uint32_t c = (&s_h[0][0])[i];
        if (c) atomicAdd(&hist[i], c);
    }
}

// One warp.  pass 0: locate the buckets of the two middle ranks; pass 1: locate the low bytes and form eta.
template <bool BF16>
__global__ void pooled_median_select_kernel(const uint32_t *__restrict__ hist, int pass, uint32_t r0, uint32_t r1,
                                            PoolState *__restrict__ st) {
    const int lane = threadIdx.x & 31;
    if (threadIdx.x >= 32) return;
    uint32_t b0, in0, b1, in1;
    if (pass == 0) {
        find_rank256(hist, r0, lane, b0, in0);
        find_rank256(hist, r1, lane, b1, in1);
        if (lane == 0) { st->bucket[0] = b0; st->inner[0] = in0; st->bucket[1] = b1; st->inner[1] = in1; }
    } else {
        find_rank256(hist, st->inner[0], lane, b0, in0);
        find_rank256(hist + 256, st->inner[1], lane, b1, in1);
        if (lane == 0) {
            const double lo = (double)widen16<BF16>(unkey16((st->bucket[0] << 8) | b0));
            const double hi = (double)widen16<BF16>(unkey16((st->bucket[1] << 8) | b1));
            st->eta = __fadd_rn((float)__ddiv_rn(__dadd_rn(lo, hi), 2.0), 0.0f);
        }
    }
}

template <bool BF16>
__global__ void __launch_bounds__(256) pooled_minmax_kernel(const uint16_t *__restrict__ x, long long M8, PoolState *__restrict__ st) {
    float lo = INFINITY, hi = -INFINITY;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < M8; i += stride) {
        float f[8];
        widen8<BF16>(__ldg(reinterpret_cast<const uint4 *>(x) + i), f);
#pragma unroll
        for (int j = 0; j < 8; ++j) { lo = fminf(lo, f[j]); hi = fmaxf(hi, f[j]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicMin(&st->lo_key, ordered_int(lo));
        atomicMax(&st->hi_key, ordered_int(hi));
    }
}

// Pooled histogram with the per-channel bin arithmetic (binary32, every operation rounded separately).
template <bool BF16>
__global__ void __launch_bounds__(256) pooled_hist_kernel(const uint16_t *__restrict__ x, long long M8, int nbins,
                                                          const PoolState *__restrict__ st, uint32_t *__restrict__ hist) {
    __shared__ uint32_t s_h[2048];
    for (int i = threadIdx.x; i < nbins; i += blockDim.x) s_h[i] = 0;
    const float lo = from_ordered_int(st->lo_key), hi = from_ordered_int(st->hi_key);
    const float scale = hi != lo ? __fdiv_rn((float)nbins, __fsub_rn(hi, lo)) : 0.0f;
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    if (hi != lo)
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < M8; i += stride) {
            float f[8];
            widen8<BF16>(__ldg(reinterpret_cast<const uint4 *>(x) + i), f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                int b = (int)floorf(__fmul_rn(__fsub_rn(f[j], lo), scale));
                b = min(max(b, 0), nbins - 1);
                atomicAdd(&s_h[b], 1u);
            }
        }
    __syncthreads();
    for (int i = threadIdx.x; i < nbins; i += blockDim.x)
        if (s_h[i]) atomicAdd(&hist[i], s_h[i]);
}

// One warp: lowest bin with the largest count -> eta = lo + (i + 1/2) * (hi - lo) / nbins.
__global__ void pooled_argmax_kernel(const uint32_t *__restrict__ hist, int nbins, PoolState *__restrict__ st) {
    const int lane = threadIdx.x & 31;
    if (threadIdx.x >= 32) return;
    uint32_t best_cnt = 0;
    int best_i = 0;
    for (int i = lane; i < nbins; i += 32) {
        const uint32_t c = hist[i];
        if (c > best_cnt) { best_cnt = c; best_i = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const uint32_t oc = __shfl_xor_sync(0xffffffffu, best_cnt, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
        if (oc > best_cnt || (oc == best_cnt && oi < best_i)) { best_cnt = oc; best_i = oi; }
    }
    if (lane == 0) {
        const float lo = from_ordered_int(st->lo_key), hi = from_ordered_int(st->hi_key);
        float mv = lo;
        if (hi != lo) {
            const float w = __fmul_rn(__fsub_rn(hi, lo), __fdiv_rn(1.0f, (float)nbins));
            mv = __fadd_rn(lo, __fmul_rn(__fadd_rn((float)best_i, 0.5f), w));
        }
        st->eta = mv;
    }
}

__global__ void init_pool_state_kernel(PoolState *st) {
    st->lo_key = 0x7fffffff;
    st->hi_key = (int)0x80000000;
    st->eta = 0.0f;
}

struct CalLayout {
    size_t hist, state, pool, pool_hist, zeroed, col_sum, total;  // hist: 3 passes x 2 x RADIX_BINS counters
};
static CalLayout cal_layout(int K) {
    CalLayout L;
    L.hist = 0;
    L.state = align_up(sizeof(uint32_t) * 3 * 2 * RADIX_BINS, 256);
    L.pool = L.state + 256;                                   // PoolState
    L.pool_hist = L.pool + 256;                               // 2048 bins, then 256 + 512 key counters
    L.zeroed = L.pool_hist + sizeof(uint32_t) * (2048 + 768);  // everything before this is cleared per call
    L.col_sum = align_up(L.zeroed, 256);                      // K column sums (binary64)
    L.total = L.col_sum + align_up(sizeof(double) * (size_t)K, 256);
    return L;
}

// m_out by an estimator other than the per-channel histogram (estimator: 0 histogram, 1 mean, 2 median; scalar: one
// eta from the pooled tensor, broadcast to the K entries of m_out).
template <bool BF16>
static cudaError_t estimate_mode(const uint16_t *x, int T, int K, int estimator, bool scalar, int nbins, float *m_out,
                                 unsigned char *ws, const CalLayout &L, cudaStream_t st) {
    PoolState *pool = reinterpret_cast<PoolState *>(ws + L.pool);
    uint32_t *phist = reinterpret_cast<uint32_t *>(ws + L.pool_hist);
    double *col_sum = reinterpret_cast<double *>(ws + L.col_sum);
    const long long M = (long long)T * K, M8 = M / 8;
    const int grid = sm_count() * 4;
    cudaError_t e = cudaSuccess;
    if (!scalar && estimator == 3) {
        static SmemOptIn opt_in_kde;
        e = ensure_dynamic_smem(kde_kernel<BF16>, 8 * KDE_MAX_T * 4, opt_in_kde);
        if (e != cudaSuccess) return e;
        return launch(kde_kernel<BF16>, dim3(K / 8), dim3(256), (size_t)8 * T * 4, st, false, x, T, K, nbins, m_out);
    }
    if (!scalar) {
        if (estimator == 1) return launch(mean_kernel<BF16>, dim3((K + 31) / 32), dim3(256), 0, st, false, x, T, K, m_out, (double *)nullptr);
        static SmemOptIn opt_in;
        const size_t smem = (size_t)3 * CW * 256 * 4;
        e = ensure_dynamic_smem(median_kernel<BF16>, (int)smem, opt_in);
        if (e != cudaSuccess) return e;
        return launch(median_kernel<BF16>, dim3((K + CW - 1) / CW), dim3(CAL_THREADS), smem, st, false, x, T, K, m_out);
    }
    if (estimator == 1) {
        e = launch(mean_kernel<BF16>, dim3((K + 31) / 32), dim3(256), 0, st, false, x, T, K, (float *)nullptr, col_sum);
        if (e != cudaSuccess) return e;
        e = launch(eta_mean_kernel, dim3(1), dim3(256), 0, st, false, (const double *)col_sum, T, K, &pool->eta);
    } else if (estimator == 2) {
        const uint32_t r0 = (uint32_t)((M - 1) / 2), r1 = (uint32_t)(M / 2);
        e = launch(pooled_key_hist_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, M8, 0, (const PoolState *)pool, phist + 2048);
        if (e != cudaSuccess) return e;
        e = launch(pooled_median_select_kernel<BF16>, dim3(1), dim3(32), 0, st, false, (const uint32_t *)(phist + 2048), 0, r0, r1, pool);
        if (e != cudaSuccess) return e;
        e = launch(pooled_key_hist_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, M8, 1, (const PoolState *)pool, phist + 2048 + 256);
        if (e != cudaSuccess) return e;
        e = launch(pooled_median_select_kernel<BF16>, dim3(1), dim3(32), 0, st, false, (const uint32_t *)(phist + 2048 + 256), 1, r0, r1, pool);
    } else {
        e = launch(init_pool_state_kernel, dim3(1), dim3(1), 0, st, false, pool);
        if (e != cudaSuccess) return e;
        if (nbins > 0) {
            e = launch(pooled_minmax_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, M8, pool);
            if (e != cudaSuccess) return e;
            e = launch(pooled_hist_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, M8, nbins, (const PoolState *)pool, phist);
            if (e != cudaSuccess) return e;
            e = launch(pooled_argmax_kernel, dim3(1), dim3(32), 0, st, false, (const uint32_t *)phist, nbins, pool);
        }
    }
    if (e != cudaSuccess) return e;
    return launch(broadcast_kernel, dim3((K + 255) / 256), dim3(256), 0, st, false, m_out, K, (const float *)&pool->eta);
}

template <bool BF16>
static scap_status calibrate_t(const uint16_t *x, int T, int K, double sparsity, int estimator, bool scalar, int nbins,
                               float *m_out, float *tau_out, unsigned char *ws, cudaStream_t st) {
    const CalLayout L = cal_layout(K);
    uint32_t *hist = reinterpret_cast<uint32_t *>(ws + L.hist);
    SelState *state = reinterpret_cast<SelState *>(ws + L.state);
    const long long M = (long long)T * K;
    const bool want_tau = sparsity > 0.0;
    const bool pdl = g_tune.pdl != 0;
    cudaError_t e = cudaMemsetAsync(ws, 0, L.zeroed, st);
    if (e != cudaSuccess) return cuda_status(e);
    const bool own_mode = estimator == 0 && !scalar;  // the strip kernel estimates the per-channel histogram mode itself
    if (!own_mode) {
        e = estimate_mode<BF16>(x, T, K, estimator, scalar, nbins, m_out, ws, L, st);
        if (e != cudaSuccess) return cuda_status(e);
        if (!want_tau) return cuda_status(launch(set_float_kernel, dim3(1), dim3(1), 0, st, false, tau_out, 0.0f));
    }
    const int HW = (nbins + 1) / 2;
    const int cw = g_tune.cal_strip;  // 16 or 32 channels per CTA
    size_t smem = (size_t)cw * HW * 4;
    if (smem < (size_t)4 * RADIX_BINS * 4) smem = (size_t)4 * RADIX_BINS * 4;  // the four copies of the first radix histogram
    static SmemOptIn opt_in32, opt_in16;
    const float *given = own_mode ? (const float *)nullptr : (const float *)m_out;
    if (cw == 16) {
        e = ensure_dynamic_smem(mode_kernel<BF16, 16>, 2048 / 2 * 16 * 4, opt_in16);
        if (e != cudaSuccess) return cuda_status(e);
        e = launch(mode_kernel<BF16, 16>, dim3((K + 15) / 16), dim3(256), smem, st, pdl, x, T, K, nbins, m_out, hist,
                   want_tau ? 1 : 0, given);
    } else {
        e = ensure_dynamic_smem(mode_kernel<BF16, 32>, 2048 / 2 * 32 * 4, opt_in32);
        if (e != cudaSuccess) return cuda_status(e);
        e = launch(mode_kernel<BF16, 32>, dim3((K + 31) / 32), dim3(512), smem, st, pdl, x, T, K, nbins, m_out, hist,
                   want_tau ? 1 : 0, given);
    }
    if (e != cudaSuccess) return cuda_status(e);
    if (!want_tau) return cuda_status(launch(set_float_kernel, dim3(1), dim3(1), 0, st, false, tau_out, 0.0f));

    const double pos = sparsity * (double)(M - 1);
    long long j = (long long)floor(pos);
    if (j > M - 1) j = M - 1;
    const double frac = pos - (double)j;
    const long long j1 = j + 1 < M ? j + 1 : M - 1;
    // radix passes: 256 channels per CTA column, enough row slabs for about four CTAs per SM
    const int gx = (K + 255) / 256;
    int gy = (sm_count() * 4 + gx - 1) / gx;
    if (gy > (T + 7) / 8) gy = (T + 7) / 8;
    const dim3 grid(gx, gy < 1 ? 1 : gy);
    // pass A (bits 30..20) was accumulated by mode_kernel; each later pass first extends the prefixes from the
    // counters of the pass before it
    e = launch(radix_pass_kernel<BF16>, grid, dim3(256), 0, st, pdl, x, (const float *)m_out, T, K, (const uint32_t *)hist, 0,
               11, (const SelState *)nullptr, (uint32_t)j, (uint32_t)j1, state, 9, 11, hist + 2 * RADIX_BINS);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(radix_pass_kernel<BF16>, grid, dim3(256), 0, st, pdl, x, (const float *)m_out, T, K,
               (const uint32_t *)(hist + 2 * RADIX_BINS), 1, 11, (const SelState *)state, 0u, 0u, state + 1, 0, 9,
               hist + 4 * RADIX_BINS);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(select_kernel, dim3(1), dim3(256), 0, st, pdl, (const uint32_t *)(hist + 4 * RADIX_BINS), 512, 9,
               (const SelState *)(state + 1), frac, tau_out);
    return cuda_status(e);
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_calibrate_workspace(int T, int K, int nbins) {
    if (T < 1 || K < 1 || nbins < 0 || nbins > 2048) return 0;
    return cal_layout(K).total;
}

scap_status scap_calibrate_ex(const void *x_calib, int T, int K, scap_dtype dt, double sparsity, scap_mode_estimator estimator,
                              scap_eta_scope scope, int nbins, float *m_out, float *tau_out, void *ws, size_t ws_bytes,
                              scap_stream_t stream) {
    if (!x_calib || !m_out || !tau_out || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (T < 1 || T > 65535 || K < 1 || (long long)T * K >= (1ll << 31)) return SCAP_ERR_SHAPE;
    if (nbins < 0 || nbins > 2048 || !(sparsity < 1.0)) return SCAP_ERR_INVALID_ARG;
    if ((int)estimator < 0 || (int)estimator > 3 || (int)scope < 0 || (int)scope > 1) return SCAP_ERR_INVALID_ARG;
    if (estimator == SCAP_MODE_KDE) {  // per channel only; the strip must fit in shared memory; nbins = grid points
        if (scope != SCAP_ETA_PER_CHANNEL || nbins < 2) return SCAP_ERR_INVALID_ARG;
        if (T > KDE_MAX_T) return SCAP_ERR_SHAPE;
    }
    if (K % 8 != 0 || !aligned16(x_calib) || !aligned16(m_out) || !aligned16(ws)) return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_calibrate_workspace(T, K, nbins)) return SCAP_ERR_WORKSPACE;
    scap_status st = check_device();
    if (st != SCAP_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned char *w = static_cast<unsigned char *>(ws);
    const uint16_t *x = static_cast<const uint16_t *>(x_calib);
    const bool scalar = scope == SCAP_ETA_SCALAR;
    return dt == SCAP_BF16 ? calibrate_t<true>(x, T, K, sparsity, (int)estimator, scalar, nbins, m_out, tau_out, w, s)
                           : calibrate_t<false>(x, T, K, sparsity, (int)estimator, scalar, nbins, m_out, tau_out, w, s);
}

scap_status scap_calibrate(const void *x_calib, int T, int K, scap_dtype dt, double sparsity, int nbins, float *m_out,
                           float *tau_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!x_calib || !m_out || !tau_out || !ws) return SCAP_ERR_INVALID_ARG;
    if (dt != SCAP_F16 && dt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (T < 1 || T > 65535 || K < 1 || (long long)T * K >= (1ll << 31)) return SCAP_ERR_SHAPE;
    if (nbins < 0 || nbins > 2048 || !(sparsity < 1.0)) return SCAP_ERR_INVALID_ARG;
    if (K % 8 != 0 || !aligned16(x_calib) || !aligned16(m_out) || !aligned16(ws)) return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_calibrate_workspace(T, K, nbins)) return SCAP_ERR_WORKSPACE;
    scap_status st = check_device();
    if (st != SCAP_OK) return st;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned char *w = static_cast<unsigned char *>(ws);
    const uint16_t *x = static_cast<const uint16_t *>(x_calib);
    return dt == SCAP_BF16 ? calibrate_t<true>(x, T, K, sparsity, 0, false, nbins, m_out, tau_out, w, s)
                           : calibrate_t<false>(x, T, K, sparsity, 0, false, nbins, m_out, tau_out, w, s);
}

}  // extern "C"
