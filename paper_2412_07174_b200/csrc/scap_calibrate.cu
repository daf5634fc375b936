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
    int valid = 0;
#pragma unroll
    for (int u = 0; u < CAL_U; ++u) {
        const int t = t0 + u * CAL_ROWS;
        v[u] = make_uint4(0, 0, 0, 0);
        if (t < T) {
            v[u] = __ldg(reinterpret_cast<const uint4 *>(xp + (size_t)t * K));
            valid = u + 1;
        }
    }
    return valid;
}

// One CTA per strip of CW channels: min/max, histogram, arg-max -> m; then the first radix histogram
// (bits 30..20 of |x - m|) of the strip is added to hist_a.
template <bool BF16>
__global__ void __launch_bounds__(CAL_THREADS) mode_kernel(const uint16_t *__restrict__ x, int T, int K, int nbins,
                                                           float *__restrict__ m_out, uint32_t *__restrict__ hist_a,
                                                           int want_hist) {
    extern __shared__ __align__(16) uint32_t smem[];
    __shared__ float s_lo[CW], s_hi[CW], s_m[CW];
    const int tid = threadIdx.x, q = tid & 3, rl = tid >> 2;
    const int k0 = blockIdx.x * CW;
    const int kc = k0 + q * 8;
    const bool ok = kc < K;  // K is a multiple of 8
    const uint16_t *xp = x + kc;
    // Up to CAL_ROWS * CAL_U = 2048 rows: the strip is read once, all loads in flight together, and the three
    // passes below run from registers; longer inputs are re-read per pass (from L2 when they fit).
    const bool resident = T <= CAL_ROWS * CAL_U;
    uint4 v[CAL_U];
    int nv = 0;
    if (resident && ok) nv = load_rows(xp, K, T, rl, v);

    if (nbins > 0) {
        // ---- pass 1: per-channel min / max
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
        float *s_mm = reinterpret_cast<float *>(smem);  // [2][CAL_ROWS][CW]
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            s_mm[rl * CW + q * 8 + j] = lo[j];
            s_mm[(CAL_ROWS + rl) * CW + q * 8 + j] = hi[j];
        }
        __syncthreads();
        if (tid < CW) {
            float l = INFINITY, h = -INFINITY;
            for (int r = 0; r < CAL_ROWS; ++r) { l = fminf(l, s_mm[r * CW + tid]); h = fmaxf(h, s_mm[(CAL_ROWS + r) * CW + tid]); }
            s_lo[tid] = l;
            s_hi[tid] = h;
        }
        __syncthreads();
        // ---- pass 2: histogram; two 16-bit counters per word (a count never exceeds T <= 65535)
        const int HW = (nbins + 1) / 2;
        for (int i = tid; i < CW * HW; i += CAL_THREADS) smem[i] = 0;
        float scale[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            lo[j] = s_lo[q * 8 + j];
            hi[j] = s_hi[q * 8 + j];
            scale[j] = hi[j] != lo[j] ? __fdiv_rn((float)nbins, __fsub_rn(hi[j], lo[j])) : 0.0f;
        }
        __syncthreads();
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
                            if (hi[j] != lo[j]) {
                                int i = (int)floorf(__fmul_rn(__fsub_rn(f[j], lo[j]), scale[j]));
                                i = min(max(i, 0), nbins - 1);
                                atomicAdd(&smem[(q * 8 + j) * HW + (i >> 1)], 1u << ((i & 1) * 16));
                            }
                        }
                    }
                }
            }
        __syncthreads();
        // ---- arg-max: lowest bin with the largest count; warp w takes channels 2w, 2w+1
        const int lane = tid & 31, warp = tid >> 5;
        for (int c = warp * (CW / (CAL_THREADS / 32)); c < (warp + 1) * (CW / (CAL_THREADS / 32)); ++c) {
            uint32_t best_cnt = 0;
            int best_i = 0;
            for (int i = lane; i < nbins; i += 32) {
                const uint32_t cnt = (smem[c * HW + (i >> 1)] >> ((i & 1) * 16)) & 0xffffu;
                if (cnt > best_cnt) { best_cnt = cnt; best_i = i; }  // ascending i: first maximum kept
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const uint32_t oc = __shfl_xor_sync(0xffffffffu, best_cnt, o);
                const int oi = __shfl_xor_sync(0xffffffffu, best_i, o);
                if (oc > best_cnt || (oc == best_cnt && oi < best_i)) { best_cnt = oc; best_i = oi; }
            }
            if (lane == 0) {
                const float l = s_lo[c], h = s_hi[c];
                float mv = l;
                if (h != l) {
                    const float w = __fmul_rn(__fsub_rn(h, l), __fdiv_rn(1.0f, (float)nbins));
                    mv = __fadd_rn(l, __fmul_rn(__fadd_rn((float)best_i, 0.5f), w));
                }
                s_m[c] = mv;
                if (k0 + c < K) m_out[k0 + c] = mv;
            }
        }
        __syncthreads();
    } else {
        if (tid < CW) {
            s_m[tid] = 0.0f;
            if (k0 + tid < K) m_out[k0 + tid] = 0.0f;
        }
        __syncthreads();
    }
    if (!want_hist) return;
    // ---- pass 3: first radix histogram of the importance |x - m|
    for (int i = tid; i < RADIX_BINS; i += CAL_THREADS) smem[i] = 0;
    float mk[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) mk[j] = s_m[q * 8 + j];
    __syncthreads();
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
                        atomicAdd(&smem[key >> 20], 1u);
                    }
                }
            }
        }
    __syncthreads();
    for (int i = tid; i < RADIX_BINS; i += CAL_THREADS)
        if (smem[i]) atomicAdd(&hist_a[i], smem[i]);
}

// Later radix passes: histogram of the next `width` key bits over the elements whose higher bits equal
// the prefix of order statistic j (hist[0]) or j+1 (hist[1]).
template <bool BF16>
__global__ void __launch_bounds__(256) radix_pass_kernel(const uint16_t *__restrict__ x, const float *__restrict__ m, long long M8,
                                                         int K, const SelState *__restrict__ st, int shift, int width,
                                                         uint32_t *__restrict__ hist) {
    __shared__ uint32_t s_h[2][RADIX_BINS];
    for (int i = threadIdx.x; i < 2 * RADIX_BINS; i += blockDim.x) (&s_h[0][0])[i] = 0;
    const uint32_t p0 = st->prefix[0], p1 = st->prefix[1];
    const uint32_t mask = (1u << width) - 1u;
    __syncthreads();
    constexpr int RU = 4;  // 16-byte loads in flight per thread
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < M8; i0 += stride * RU) {
        uint4 v[RU];
        float4 ma[RU], mb[RU];
#pragma unroll
        for (int u = 0; u < RU; ++u) {
            const long long i = i0 + stride * u;
            v[u] = make_uint4(0, 0, 0, 0);
            ma[u] = mb[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < M8) {
                v[u] = __ldg(reinterpret_cast<const uint4 *>(x) + i);
                const int kc = (int)((i * 8) % K);
                ma[u] = __ldg(reinterpret_cast<const float4 *>(m + kc));
                mb[u] = __ldg(reinterpret_cast<const float4 *>(m + kc + 4));
            }
        }
#pragma unroll
        for (int u = 0; u < RU; ++u) {
            if (i0 + stride * u < M8) {
                float f[8];
                widen8<BF16>(v[u], f);
                const float mk[8] = {ma[u].x, ma[u].y, ma[u].z, ma[u].w, mb[u].x, mb[u].y, mb[u].z, mb[u].w};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t key = __float_as_uint(__fsub_rn(f[j], mk[j])) & 0x7fffffffu;
                    const uint32_t hi = key >> (shift + width);
                    const uint32_t b = (key >> shift) & mask;
                    if (hi == p0) atomicAdd(&s_h[0][b], 1u);
                    if (hi == p1) atomicAdd(&s_h[1][b], 1u);
                }
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * RADIX_BINS; i += blockDim.x) {
        const uint32_t v = (&s_h[0][0])[i];
        if (v) atomicAdd(&hist[i], v);
    }
}

// One CTA.  Warp w (0 or 1) finds the bucket holding its order statistic in hist[first ? 0 : w], extends
// the prefix by `width` bits and rebases the rank.  After the last pass thread 0 interpolates:
// tau = v_j + frac * (v_j1 - v_j) in binary64, each operation rounded once, then rounded to binary32.
__global__ void select_kernel(const uint32_t *__restrict__ hist, int nb, int width, int first, int last, uint32_t j,
                              uint32_t j1, double frac, SelState *__restrict__ st, float *__restrict__ tau_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __shared__ uint32_t s_cnt[2][RADIX_BINS];  // the counts, fetched with all loads in flight (the scan below is serial)
    for (int i = threadIdx.x; i < 2 * nb; i += blockDim.x) {
        const int w = i / nb, b = i - w * nb;
        s_cnt[w][b] = hist[(first ? 0 : w * RADIX_BINS) + b];
    }
    __syncthreads();
    if (warp < 2) {
        const uint32_t *h = s_cnt[warp];
        const uint32_t rank = first ? (warp == 0 ? j : j1) : st->rank[warp];
        const uint32_t prefix = first ? 0u : st->prefix[warp];
        uint32_t carry = 0, found_b = 0, found_r = 0;
        bool found = false;
        for (int c0 = 0; c0 < nb && !found; c0 += 32) {
            const uint32_t cnt = (c0 + lane < nb) ? h[c0 + lane] : 0u;
            uint32_t v = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += t;
            }
            const uint32_t incl = carry + v, excl = incl - cnt;
            const unsigned hit = __ballot_sync(0xffffffffu, rank >= excl && rank < incl);
            if (hit) {
                const int src = __ffs(hit) - 1;
                found_b = (uint32_t)(c0 + src);
                found_r = rank - __shfl_sync(0xffffffffu, excl, src);
                found = true;
            }
            carry = __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            st->prefix[warp] = (prefix << width) | found_b;
            st->rank[warp] = found_r;
        }
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        const double vj = (double)__uint_as_float(st->prefix[0]);
        const double vj1 = (double)__uint_as_float(st->prefix[1]);
        const double t64 = __dadd_rn(vj, __dmul_rn(frac, __dsub_rn(vj1, vj)));
        *tau_out = (float)t64;
    }
}

__global__ void set_float_kernel(float *p, float v) { *p = v; }

struct CalLayout {
    size_t hist, state, total;  // hist: 3 passes x 2 x RADIX_BINS counters
};
static CalLayout cal_layout() {
    CalLayout L;
    L.hist = 0;
    L.state = align_up(sizeof(uint32_t) * 3 * 2 * RADIX_BINS, 256);
    L.total = L.state + 256;
    return L;
}

template <bool BF16>
static scap_status calibrate_t(const uint16_t *x, int T, int K, double sparsity, int nbins, float *m_out, float *tau_out,
                               unsigned char *ws, cudaStream_t st) {
    const CalLayout L = cal_layout();
    uint32_t *hist = reinterpret_cast<uint32_t *>(ws + L.hist);
    SelState *state = reinterpret_cast<SelState *>(ws + L.state);
    const long long M = (long long)T * K;
    const bool want_tau = sparsity > 0.0;
    cudaError_t e = cudaMemsetAsync(ws, 0, L.total, st);
    if (e != cudaSuccess) return cuda_status(e);
    const int HW = (nbins + 1) / 2;
    size_t smem = (size_t)CW * HW * 4;
    if (smem < (size_t)2 * CAL_ROWS * CW * 4) smem = (size_t)2 * CAL_ROWS * CW * 4;
    if (smem < (size_t)RADIX_BINS * 4) smem = (size_t)RADIX_BINS * 4;
    static bool attr_set[2] = {false, false};
    if (!attr_set[BF16]) {
        e = cudaFuncSetAttribute(mode_kernel<BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2048 / 2 * CW * 4);
        if (e != cudaSuccess) return cuda_status(e);
        attr_set[BF16] = true;
    }
    e = launch(mode_kernel<BF16>, dim3((K + CW - 1) / CW), dim3(CAL_THREADS), smem, st, false, x, T, K, nbins, m_out, hist,
               want_tau ? 1 : 0);
    if (e != cudaSuccess) return cuda_status(e);
    if (!want_tau) return cuda_status(launch(set_float_kernel, dim3(1), dim3(1), 0, st, false, tau_out, 0.0f));

    const double pos = sparsity * (double)(M - 1);
    long long j = (long long)floor(pos);
    if (j > M - 1) j = M - 1;
    const double frac = pos - (double)j;
    const long long j1 = j + 1 < M ? j + 1 : M - 1;
    const int grid = sm_count() * 4;
    // pass A (bits 30..20) was accumulated by mode_kernel
    e = launch(select_kernel, dim3(1), dim3(256), 0, st, false, (const uint32_t *)hist, RADIX_BINS, 11, 1, 0, (uint32_t)j,
               (uint32_t)j1, frac, state, tau_out);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(radix_pass_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, (const float *)m_out, M / 8, K,
               (const SelState *)state, 9, 11, hist + 2 * RADIX_BINS);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(select_kernel, dim3(1), dim3(256), 0, st, false, (const uint32_t *)(hist + 2 * RADIX_BINS), RADIX_BINS, 11, 0, 0,
               0u, 0u, frac, state, tau_out);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(radix_pass_kernel<BF16>, dim3(grid), dim3(256), 0, st, false, x, (const float *)m_out, M / 8, K,
               (const SelState *)state, 0, 9, hist + 4 * RADIX_BINS);
    if (e != cudaSuccess) return cuda_status(e);
    e = launch(select_kernel, dim3(1), dim3(256), 0, st, false, (const uint32_t *)(hist + 4 * RADIX_BINS), 512, 9, 0, 1, 0u, 0u,
               frac, state, tau_out);
    return cuda_status(e);
}

}  // namespace scap

using namespace scap;

extern "C" {

size_t scap_calibrate_workspace(int T, int K, int nbins) {
    if (T < 1 || K < 1 || nbins < 0 || nbins > 2048) return 0;
    return cal_layout().total;
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
    return dt == SCAP_BF16 ? calibrate_t<true>(x, T, K, sparsity, nbins, m_out, tau_out, w, s)
                           : calibrate_t<false>(x, T, K, sparsity, nbins, m_out, tau_out, w, s);
}

}  // extern "C"
