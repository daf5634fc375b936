// Sparse FC on 8-bit weights (Table 4 applies SCAP to 8-bit models).  Storage: Wq[K,N] signed 8-bit, input-channel-
// major like the 16-bit layout, one binary32 scale per input channel, W[k,n] = wscale[k] * Wq[k,n].  Because the
// scale belongs to the input channel it is folded into the pruned activation once per kept channel (d * wscale),
// and the streaming loop multiplies by the raw integers.  A kept row of a 128-column tile is 128 bytes, so a
// thread's 16-byte load covers 16 columns and 8 lanes cover the row; everything else (cluster split, ballot
// compaction, register double buffer, cluster exchange) is the FMA kernel of scap_fc.cuh.
#include <string.h>

#include "scap_fc.cuh"

namespace scap {

constexpr int Q8_TN = 128;   // columns per CTA
constexpr int Q8_CPT = 16;   // columns per thread (one 16-byte load)

// Two fp32 values in one 64-bit register, for the packed fp32 instructions of sm_100 (add.f32x2 / fma.rn.f32x2: one
// instruction per two weights; the unpack is bound by instruction issue, so this is worth a third of its time).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(__float_as_uint(lo)), "r"(__float_as_uint(hi)));
    return r;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
    unsigned long long r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float &lo, float &hi) {
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}

// acc[b][j] (pairs of columns) += xv * q for the 16 signed bytes of v.  (byte ^ 0x80) placed in the mantissa of 2^23 reads
// as 2^23 + (q + 128); adding -(2^23 + 128) gives q exactly; both steps and the multiply-add run two columns at a time.
template <int BT, int CAP>
__device__ __forceinline__ void fma_row_q8(unsigned long long (&acc)[BT][8], const uint4 &v, const float *__restrict__ s_xs, int i) {
    const uint32_t u[4] = {v.x ^ 0x80808080u, v.y ^ 0x80808080u, v.z ^ 0x80808080u, v.w ^ 0x80808080u};
    const unsigned long long neg = pack2(-8388736.0f, -8388736.0f);
    unsigned long long w[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        w[2 * q] = add2(pack2(__uint_as_float(__byte_perm(u[q], 0x4B000000u, 0x7650)), __uint_as_float(__byte_perm(u[q], 0x4B000000u, 0x7651))), neg);
        w[2 * q + 1] = add2(pack2(__uint_as_float(__byte_perm(u[q], 0x4B000000u, 0x7652)), __uint_as_float(__byte_perm(u[q], 0x4B000000u, 0x7653))), neg);
    }
#pragma unroll
    for (int b = 0; b < BT; ++b) {
        const float xv = s_xs[b * CAP + i];
        const unsigned long long x2 = pack2(xv, xv);
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[b][j] = fma2(x2, w[j], acc[b][j]);
    }
}

template <int BT, int MODE, typename XT>
__global__ void __launch_bounds__(FC_THREADS, 2) fc_q8_kernel(const FcArgs a) {
    constexpr int TNT = Q8_TN, EPI = EPI_BIAS;
    constexpr int NT = FC_THREADS, PU = fc_pu(BT), CAP = fc_cap(BT), RB = fc_rb(BT), U = fc_unroll(BT);
    constexpr int CAPC = CAP / 32;
    constexpr int LPR = TNT / Q8_CPT;  // 8 lanes per row segment
    constexpr int NR = NT / LPR;       // 32 row groups per CTA
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *s_k = reinterpret_cast<uint32_t *>(smem);
    float *s_xs = reinterpret_cast<float *>(smem) + CAP;
    float *s_red = reinterpret_cast<float *>(smem);
    float *s_gather = reinterpret_cast<float *>(smem + fc_main_bytes(BT));
    uint32_t *s_bits = reinterpret_cast<uint32_t *>(s_gather + BT * GATHER_LD);
    int *s_wcnt = reinterpret_cast<int *>(s_bits + CAPC) + 16;

    const int tile = blockIdx.x, s = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = tid / LPR, cl = tid % LPR;
    const int B = a.B, S = a.S, K = a.K;
    const XT *xg = reinterpret_cast<const XT *>(a.x);

    const int col = tile * TNT + cl * Q8_CPT;
    const bool col_ok = col < a.Nh;  // N is a multiple of 16
    const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (size_t)col;
    const size_t row_bytes = (size_t)a.ldw;

    const int per = (TNT + S - 1) / S;
    float bias0[2], bias1[2];

    unsigned long long acc2[BT][8];  // 16 columns per batch row as 8 packed pairs
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc2[b][j] = 0ull;

    const int nchunks = (K + 31) >> 5;
    const int my_chunks = nchunks > s ? (nchunks - s + S - 1) / S : 0;
    float tau = 0.0f;
    // Nothing is read before earlier work on the stream is complete: tau, m, the scales and the biases may have been
    // written by it just as the activations may; all of them are read through L2.
    griddep_wait();
    if (!a.hold_dependents) griddep_launch_dependents();
    if constexpr (MODE == MODE_GATHER) {
        float tv = 0.0f;
        if (lane == 0) tv = ld_act(a.tau);
        tau = __shfl_sync(0xffffffffu, tv, 0);
    }
    prefetch_bias<true, EPI, TNT>(a, tile, s, per, bias0, bias1);
    for (int j0 = 0; j0 < my_chunks; j0 += CAPC) {
        const int nj = min(CAPC, my_chunks - j0);
        const int pw = (nj + FC_WARPS - 1) / FC_WARPS;  // chunks per warp this fill: warp w owns chunks w * pw .. w * pw + pw - 1
        XT xraw[PU][BT];
        float xv[PU][BT], mk[PU], sc[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pw + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            mk[p] = a.m ? ld_act_if(a.m + k, p < pw && j < nj && k < K) : 0.0f;
            sc[p] = ld_act_if(a.wscale + k, p < pw && j < nj && k < K);
        }
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pw + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            const bool ok = p < pw && j < nj && k < K;
#pragma unroll
            for (int b = 0; b < BT; ++b) xraw[p][b] = ld_act_if(xg + (size_t)(b < B ? b : 0) * a.x_ld + k, ok && b < B);
        }
#pragma unroll
        for (int p = 0; p < PU; ++p)
#pragma unroll
            for (int b = 0; b < BT; ++b) xv[p][b] = widen1(xraw[p][b]);
        uint32_t km[PU];
        unsigned bal[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pw + p;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            const bool ok = p < pw && j < nj && k < K;
            uint32_t m_ = 0;
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                if constexpr (MODE == MODE_GATHER) {
                    const float dv = a.m ? __fsub_rn(xv[p][b], mk[p]) : xv[p][b];
                    xv[p][b] = dv;
                    m_ |= (ok && b < B && fabsf(dv) >= tau) ? (1u << b) : 0u;
                } else {
                    m_ = ok ? 1u : 0u;
                }
            }
            km[p] = m_;
            bal[p] = __ballot_sync(0xffffffffu, m_ != 0);
        }
        int my_off[PU], wtotal = 0;
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            my_off[p] = wtotal;
            wtotal += __popc(bal[p]);
        }
        if (lane == 0) s_wcnt[warp] = wtotal;
        if (MODE == MODE_GATHER && a.bits && tile == 0) {
            unsigned mine = 0;
#pragma unroll
            for (int p = 0; p < PU; ++p) mine = lane == p ? bal[p] : mine;
            const int j = warp * pw + lane;
            if (lane < pw && j < nj) a.bits[s + S * (j0 + j)] = mine;
        }
        __syncthreads();
        int cnt = 0, wbase = 0;
#pragma unroll
        for (int w = 0; w < FC_WARPS; ++w) {
            const int c = s_wcnt[w];
            cnt += c;
            wbase += w < warp ? c : 0;
        }
        // kept channels and their pruned values times the channel's weight scale, in ascending channel order
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            if (km[p]) {
                const int j = warp * pw + p;
                const int pos = wbase + my_off[p] + __popc(bal[p] & ((1u << lane) - 1u));
                s_k[pos] = (uint32_t)((s + S * (j0 + j)) * 32 + lane);
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    s_xs[b * CAP + pos] = (MODE == MODE_DENSE || ((km[p] >> b) & 1u)) ? __fmul_rn(xv[p][b], sc[p]) : 0.0f;
            }
        }
        __syncthreads();
        if (col_ok) {
            constexpr int G = U / 2;
            const int nrows = cnt > rg ? (cnt - rg + NR - 1) / NR : 0;
            uint4 ga[G], gb[G];
#pragma unroll
            for (int u = 0; u < G; ++u)
                if (u < nrows) ga[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * u] * row_bytes);
#pragma unroll
            for (int u = 0; u < G; ++u)
                if (G + u < nrows) gb[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (G + u)] * row_bytes);
            for (int t0 = 0; t0 < nrows; t0 += 2 * G) {
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + u < nrows) fma_row_q8<BT, CAP>(acc2, ga[u], s_xs, rg + NR * (t0 + u));
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + 2 * G + u < nrows) ga[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 2 * G + u)] * row_bytes);
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + G + u < nrows) fma_row_q8<BT, CAP>(acc2, gb[u], s_xs, rg + NR * (t0 + G + u));
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + 3 * G + u < nrows) gb[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 3 * G + u)] * row_bytes);
            }
        }
        __syncthreads();
    }

    float acc[BT][16];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int j = 0; j < 8; ++j) unpack2(acc2[b][j], acc[b][2 * j], acc[b][2 * j + 1]);
    // the four row groups of a warp (lanes l, l ^ 8, l ^ 16, l ^ 24 hold the same columns) are added by shuffles
    // in a fixed order; lanes 0-7 then hold the warp's partial of its 128 columns
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            acc[b][j] += __shfl_xor_sync(0xffffffffu, acc[b][j], 8);
            acc[b][j] += __shfl_xor_sync(0xffffffffu, acc[b][j], 16);
        }
    cg::cluster_group cluster = cg::this_cluster();
    float *owner[MAX_CLUSTER];
#pragma unroll
    for (int q = 0; q < MAX_CLUSTER; ++q) owner[q] = (S > 1 && q < S) ? cluster.map_shared_rank(s_gather, q) : s_gather;
#pragma unroll
    for (int b0 = 0; b0 < BT; b0 += RB) {
        if (lane < LPR) {
#pragma unroll
            for (int rb = 0; rb < RB; ++rb) {
                float4 *dst = reinterpret_cast<float4 *>(s_red + ((warp * RB + rb) * TNT + cl * Q8_CPT));
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    dst[q] = make_float4(acc[b0 + rb][4 * q], acc[b0 + rb][4 * q + 1], acc[b0 + rb][4 * q + 2], acc[b0 + rb][4 * q + 3]);
            }
        }
        __syncthreads();
        reduce_push_round<BT, EPI, TNT, FC_WARPS, RB>(s_red, b0, B, s, per, owner);
        __syncthreads();
    }
    if (S > 1) cluster.sync();
    else __syncthreads();
    finish_columns<true, BT, EPI, TNT>(a, tile, s, per, s_gather, bias0, bias1);
}

// Split-K factor: the most CTAs (tiles of 128 columns x S) that are all resident; ties: the larger cluster.
static int q8_split(int K, int N) {
    const int tiles = (N + Q8_TN - 1) / Q8_TN;
    int best_S = 1;
    long long best = -1;
    for (int S = 1; S <= MAX_CLUSTER; ++S) {
        if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
        if (S > 1 && K / S < 64) continue;
        const long long ctas = (long long)tiles * S;
        if (S > 1 && ctas > resident_ctas(S)) continue;
        if (ctas >= best) { best = ctas; best_S = S; }
    }
    return best_S;
}

template <int BT, int MODE, typename XT>
static cudaError_t launch_q8_t(const FcArgs &a, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_q8_kernel<BT, MODE, XT>;
    cudaError_t e0 = ensure_dynamic_smem(kern, fc_smem_bytes(BT), opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3((a.Nh + Q8_TN - 1) / Q8_TN, a.S), dim3(FC_THREADS), fc_smem_bytes(BT), a.S, st, g_tune.pdl != 0, a);
}

// xkind: 0 fp16, 1 bf16, 2 float activations.  Batches beyond two rows run two rows at a time (row results are
// independent; the union mask then spans two rows).
static cudaError_t launch_q8(int mode, int xkind, FcArgs a, cudaStream_t st) {
    const int B = a.B;
    const size_t xsz = xkind == 2 ? 4 : 2;
    const unsigned char *x0 = static_cast<const unsigned char *>(a.x);
    float *y0 = a.y;
    for (int b0 = 0; b0 < B; b0 += 2) {
        a.B = B - b0 >= 2 ? 2 : 1;
        a.x = x0 + (size_t)b0 * a.x_ld * xsz;
        a.y = y0 + (size_t)b0 * a.y_ld;
        cudaError_t e;
        if (a.B == 1) {
            if (mode == MODE_DENSE) e = xkind == 2 ? launch_q8_t<1, MODE_DENSE, float>(a, st) : xkind == 1 ? launch_q8_t<1, MODE_DENSE, __nv_bfloat16>(a, st) : launch_q8_t<1, MODE_DENSE, __half>(a, st);
            else e = xkind == 1 ? launch_q8_t<1, MODE_GATHER, __nv_bfloat16>(a, st) : launch_q8_t<1, MODE_GATHER, __half>(a, st);
        } else {
            if (mode == MODE_DENSE) e = xkind == 1 ? launch_q8_t<2, MODE_DENSE, __nv_bfloat16>(a, st) : launch_q8_t<2, MODE_DENSE, __half>(a, st);
            else e = xkind == 1 ? launch_q8_t<2, MODE_GATHER, __nv_bfloat16>(a, st) : launch_q8_t<2, MODE_GATHER, __half>(a, st);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace scap

using namespace scap;

extern "C" {

static scap_status q8_check(const void *x, const void *Wq, const float *wscale, const float *m, const float *b, float *y, int B, int K,
                            int N, scap_dtype xdt, const void *ws, size_t ws_bytes) {
    if (!x || !Wq || !wscale || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (xdt != SCAP_F16 && xdt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
    if (N % 16 != 0 || !aligned16(x) || !aligned16(Wq) || !aligned16(y) || !aligned16(ws) || (m && !aligned16(m)) || (b && !aligned16(b)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    return check_device();
}

scap_status scap_sparse_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *m,
                              const float *tau, const float *b_fused, float *y, int B, int K, int N, uint32_t *idx_out,
                              int *nnz_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!tau) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q8_check(x, Wq, wscale, m, b_fused, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    if ((idx_out || nnz_out) && B > 2) return SCAP_ERR_SHAPE;  // the kept list describes one launch (at most two rows)
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = B; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = x; a.x_ld = K; a.m = m; a.tau = tau; a.bias = b_fused; a.y = y; a.y_ld = N;
    const bool inspect = idx_out || nnz_out;
    if (inspect) a.bits = reinterpret_cast<uint32_t *>(ws);
    cudaError_t e = launch_q8(MODE_GATHER, xdt == SCAP_BF16 ? 1 : 0, a, st);
    if (e != cudaSuccess) return cuda_status(e);
    if (inspect) e = launch_expand_bits(a.bits, K, idx_out, nnz_out, st);
    return cuda_status(e);
}

scap_status scap_dense_fc_q8(const void *x, scap_dtype xdt, const signed char *Wq, const float *wscale, const float *b, float *y,
                             int B, int K, int N, void *ws, size_t ws_bytes, scap_stream_t stream) {
    scap_status stt = q8_check(x, Wq, wscale, nullptr, b, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = B; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = x; a.x_ld = K; a.bias = b; a.y = y; a.y_ld = N;
    return cuda_status(launch_q8(MODE_DENSE, xdt == SCAP_BF16 ? 1 : 0, a, reinterpret_cast<cudaStream_t>(stream)));
}

scap_status scap_fold_bias_q8(const signed char *Wq, const float *wscale, const float *m, const float *b, int K, int N,
                              float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!m) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q8_check(m, Wq, wscale, nullptr, b, b_fused, 1, K, N, SCAP_BF16, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    FcArgs a;
    memset(&a, 0, sizeof(a));
    a.W = Wq; a.wscale = wscale; a.K = K; a.ldw = N; a.Nh = N; a.B = 1; a.tn = Q8_TN; a.S = q8_split(K, N);
    a.x = m; a.x_ld = K; a.bias = b; a.y = b_fused; a.y_ld = N;
    a.hold_dependents = 1;  // it writes a parameter: ordinary stream order on both sides
    return cuda_status(launch_q8(MODE_DENSE, 2, a, reinterpret_cast<cudaStream_t>(stream)));
}

}  // extern "C"
