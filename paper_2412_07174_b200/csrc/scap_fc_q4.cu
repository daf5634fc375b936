// Sparse FC on group-wise 4-bit weights (Table 4 applies SCAP to AWQ 4-bit models).  Storage: Wq[K, N/2] bytes, two
// unsigned 4-bit codes per byte (column 2j in the low nibble of byte j), input-channel-major like the 16-bit layout;
// groups of `group` consecutive INPUT channels share, per output column, a binary32 scale and a zero point 0..15:
//     W[k,n] = scale[k / group, n] * (q[k,n] - zero[k / group, n]).
// A kept channel is still one contiguous row (N/2 bytes), but its scale and zero point belong to its group, so the
// work is laid out to stay inside a group for as long as possible:
//   - the S ranks of a cluster split the input channels into contiguous ranges of whole groups (not interleaved chunks);
//   - the kept list of a rank is ascending, and row group g of the CTA streams a contiguous stretch of it, so it meets
//     one or two groups per call; at the start of each stretch inside one group it requests that group's scales and
//     zero points for its 16 columns once (16 + 4 registers), accumulates sum d * (q - zero) over the stretch, and
//     scales the sum once: y += scale * sum.
// A thread owns 16 columns: one 8-byte load per kept row (16 codes); a code becomes a float by placing it in the mantissa
// of 2^23 and subtracting 2^23 + zero (exact).  Threshold, ballot compaction, cluster exchange and the epilogue are
// those of the 16-bit kernel (scap_fc.cuh); nothing is read before the dependency wait.
#include <string.h>
#include <type_traits>

#include "scap_fc.cuh"

namespace scap {

constexpr int Q4_TN = 128;   // columns per CTA: a row segment is 64 bytes = 8 lanes x 8 bytes (two CTAs per SM: the unpack arithmetic needs the warps)
constexpr int Q4_CPT = 16;   // columns per thread (one 8-byte load)
__host__ __device__ constexpr int q4_unroll(int BT) { return BT <= 1 ? 16 : 8; }  // row loads in flight per thread
constexpr int Q4_MAXG = 64;  // most groups per fill (2048 channels of 32)
// list region, overlaid by the reduction buffer of the row groups
__host__ __device__ constexpr int q4_main_bytes(int BT) {
    const int red = (FC_THREADS / (Q4_TN / Q4_CPT)) * fc_rb(BT) * Q4_TN * 4;
    return fc_main_bytes(BT) > red ? fc_main_bytes(BT) : red;
}

struct Q4Args {
    FcArgs f;                    // W = Wq; ldw = N (columns); the rest as in the 16-bit kernel
    const float *scale;          // [ceil(K / group), N]
    const unsigned char *zero;   // [ceil(K / group), N]
    int group;                   // input channels per group: a multiple of 32
};

__device__ __forceinline__ uint2 ld_stream8_if(const void *p, bool on) {
    uint2 v;
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %3, 0; mov.u32 %0, 0; mov.u32 %1, 0; @q ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2]; }"
                 : "=r"(v.x), "=r"(v.y) : "l"(p), "r"((unsigned)on));
    return v;
}

// acc[j] (pairs of columns) += xv * q_j for the 16 codes of v.  The zero point is not subtracted per weight: over the rows
// of one group sum xv (q - z) = sum xv q - z sum xv, and the second sum is one addition per row (the caller keeps it).
// A code becomes a float by placing it in the mantissa of 2^23 and subtracting 2^23 (exact); the even and the odd codes
// of a word are masked out together, then one byte permute per code; subtraction and multiply-add run two columns at a time.
__device__ __forceinline__ void fma_row_q4(unsigned long long (&acc)[8], const uint2 &v, float xv) {
    const unsigned long long neg = pack2(-8388608.0f, -8388608.0f);
    const unsigned long long x2 = pack2(xv, xv);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t w = h ? v.y : v.x;
        const uint32_t ev = w & 0x0F0F0F0Fu, od = (w >> 4) & 0x0F0F0F0Fu;  // codes 0,2,4,6 and 1,3,5,7, one per byte
        const unsigned long long q01 = add2(pack2(__uint_as_float(__byte_perm(ev, 0x4B000000u, 0x7650)), __uint_as_float(__byte_perm(od, 0x4B000000u, 0x7650))), neg);
        const unsigned long long q23 = add2(pack2(__uint_as_float(__byte_perm(ev, 0x4B000000u, 0x7651)), __uint_as_float(__byte_perm(od, 0x4B000000u, 0x7651))), neg);
        const unsigned long long q45 = add2(pack2(__uint_as_float(__byte_perm(ev, 0x4B000000u, 0x7652)), __uint_as_float(__byte_perm(od, 0x4B000000u, 0x7652))), neg);
        const unsigned long long q67 = add2(pack2(__uint_as_float(__byte_perm(ev, 0x4B000000u, 0x7653)), __uint_as_float(__byte_perm(od, 0x4B000000u, 0x7653))), neg);
        acc[4 * h + 0] = fma2(x2, q01, acc[4 * h + 0]);
        acc[4 * h + 1] = fma2(x2, q23, acc[4 * h + 1]);
        acc[4 * h + 2] = fma2(x2, q45, acc[4 * h + 2]);
        acc[4 * h + 3] = fma2(x2, q67, acc[4 * h + 3]);
    }
}

// PUT = chunk slots per warp and fill that the threshold code is unrolled for (at most fc_pu(BT), which sizes the list):
// that code is bound by instruction issue, so the launcher picks the smallest instantiation whose fill still holds a
// whole group and the rank's channels.
template <int BT, int MODE, typename XT, int PUT = fc_pu(BT)>
__global__ void __launch_bounds__(FC_THREADS, 2) fc_q4_kernel(const Q4Args qa) {
    const FcArgs &a = qa.f;
    constexpr int TNT = Q4_TN, EPI = EPI_BIAS, U = q4_unroll(BT);
    constexpr int PU = PUT, CAP = fc_cap(BT), RB = fc_rb(BT);
    constexpr int FILL = FC_WARPS * PU * 32;  // channels per fill
    static_assert(PUT >= 1 && PUT <= fc_pu(BT), "the list is sized for fc_pu(BT) slots per warp");
    constexpr int LPR = TNT / Q4_CPT;      // 8 lanes per row segment
    constexpr int NR = FC_THREADS / LPR;   // 32 row groups per CTA
    static_assert(RB == BT, "one reduction round");
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *s_k = reinterpret_cast<uint32_t *>(smem);
    float *s_xs = reinterpret_cast<float *>(smem) + CAP;
    float *s_red = reinterpret_cast<float *>(smem);
    float *s_gather = reinterpret_cast<float *>(smem + q4_main_bytes(BT));
    int *s_wcnt = reinterpret_cast<int *>(s_gather + BT * GATHER_LD);
    int *s_goff = s_wcnt + FC_WARPS;       // [groups of the fill + 1]: list position of each group's first kept channel

    const int tile = blockIdx.x, s = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = tid / LPR, cl = tid % LPR;
    const int B = a.B, S = a.S, K = a.K, N = a.ldw, group = qa.group;
    const XT *xg = reinterpret_cast<const XT *>(a.x);

    const int col = tile * TNT + cl * Q4_CPT;
    const bool col_ok = col < N;  // N is a multiple of 16
    const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (size_t)col / 2;
    const size_t row_bytes = (size_t)N / 2;
    const int per = (TNT + S - 1) / S;

    float y_acc[BT][16];
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
        for (int j = 0; j < 16; ++j) y_acc[b][j] = 0.0f;

    // this rank's contiguous range of whole groups
    const int G = (K + group - 1) / group, gper = (G + S - 1) / S;
    const int g_lo = min(G, s * gper), g_hi = min(G, g_lo + gper);
    const int cpg = group >> 5;            // chunks per group
    const int fill_groups = FILL / group;  // whole groups per fill (the launcher guarantees at least one)

    // The barrier the split-K partials of this rank's columns will land on (asynchronous exchange, as in the 16-bit kernel)
    const uint32_t bar = smem_addr(s_goff + Q4_MAXG + 2);
    if (S > 1) {
        if (tid == 0) {
            const int owned = max(0, min(per, TNT - s * per));
            mbarrier_init(bar, 1);
            mbarrier_arrive_expect(bar, (uint32_t)(S * B * owned * 4));
        }
        cluster_arrive_relaxed();
    }
    griddep_wait();  // nothing is read before earlier work on the stream is complete
    if (!a.hold_dependents) griddep_launch_dependents();
    // tau: one request per CTA, issued first and handed to the other warps through shared memory once the activation
    // requests of the first fill are out (as in the 16-bit kernel: the two round trips to L2 overlap)
    float tau = 0.0f, tau_reg = 0.0f;
    if (MODE == MODE_GATHER && tid == 0) tau_reg = ld_act(a.tau);
    float bias0[2], bias1[2];
    bool first_fill = true;

    for (int g0 = g_lo; g0 < g_hi; g0 += fill_groups) {
        const int ng = min(fill_groups, g_hi - g0);         // groups of this fill
        const int k0 = g0 * group;                          // first channel of the fill
        const int nj = min((ng * group) >> 5, ((K - k0) + 31) >> 5);  // chunks of the fill
        const int pw = (nj + FC_WARPS - 1) / FC_WARPS;      // consecutive chunks per warp
        // ---- threshold: as in the 16-bit kernel, with the rank's chunks contiguous
        // (addresses and predicates first, then all requests of the lane back to back: the code runs on every warp of the
        // SM at the same moment and is bound by instruction issue)
        const int nw = max(0, min(pw, nj - warp * pw));      // chunks of this warp
        const int kbase = k0 + warp * pw * 32 + lane;        // this lane's channel in the warp's first chunk
        const XT *xrow[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) xrow[b] = xg + (size_t)(b < B ? b : 0) * a.x_ld + kbase;
        const float *mrow = (MODE == MODE_GATHER && a.m) ? a.m + kbase : nullptr;
        bool okx[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) okx[p] = p < nw && kbase + p * 32 < K;
        XT xraw[PU][BT];
        float xv[PU][BT], mk[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
#pragma unroll
            for (int b = 0; b < BT; ++b) xraw[p][b] = ld_act_if(xrow[b] + p * 32, okx[p] && b < B);
        }
#pragma unroll
        for (int p = 0; p < PU; ++p) mk[p] = ld_act_if(mrow + p * 32, mrow != nullptr && okx[p]);
        if (first_fill) {
            if constexpr (MODE == MODE_GATHER) {
                float *s_tau = reinterpret_cast<float *>(s_goff + Q4_MAXG + 1);
                if (tid == 0) *s_tau = tau_reg;
                __syncthreads();
                tau = *s_tau;
            }
            prefetch_bias<true, EPI, TNT>(a, tile, s, per, bias0, bias1);  // behind the activation requests
            first_fill = false;
        }
        uint32_t km[PU];
        unsigned bal[PU];
        int my_off[PU], wtotal = 0;
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const bool ok = okx[p];
            uint32_t m_ = 0;
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                xv[p][b] = widen1(xraw[p][b]);
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
            my_off[p] = wtotal;
            wtotal += __popc(bal[p]);
        }
        if (lane == 0) s_wcnt[warp] = wtotal;
        if (MODE == MODE_GATHER && a.bits && tile == 0) {
            unsigned mine = 0;
#pragma unroll
            for (int p = 0; p < PU; ++p) mine = lane == p ? bal[p] : mine;
            const int j = warp * pw + lane;
            if (lane < pw && j < nj) a.bits[(k0 >> 5) + j] = mine;
        }
        __syncthreads();
        int cnt = 0, wbase = 0;
#pragma unroll
        for (int w = 0; w < FC_WARPS; ++w) {
            const int c = s_wcnt[w];
            cnt += c;
            wbase += w < warp ? c : 0;
        }
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = warp * pw + p;
            if (lane == 0 && p < pw && j < nj && j % cpg == 0) s_goff[j / cpg] = wbase + my_off[p];  // the chunk opens a group
            if (km[p]) {
                const int pos = wbase + my_off[p] + __popc(bal[p] & ((1u << lane) - 1u));
                s_k[pos] = (uint32_t)(kbase + p * 32);
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    s_xs[b * CAP + pos] = (MODE == MODE_DENSE || ((km[p] >> b) & 1u)) ? xv[p][b] : 0.0f;
            }
        }
        if (tid == 0) s_goff[ng] = cnt;
        __syncthreads();

        // ---- stream: a WARP takes a contiguous range [r_lo, r_hi) of the list and its four row groups take every fourth
        // position of it (row group j the positions = r_lo + j mod 4), so that all lanes of the warp meet the group
        // boundaries in the same iteration and run the same number of rounds (with a contiguous range per row group
        // the four ranges of a warp crossed their boundaries at different places and the warp ran up to twice the rounds).
        // Inside the range: one stretch per group.  Shorter lists (fewer than 24 rows per row group) keep a contiguous range
        // per row group instead: there every row group of the interleaved form would open and close every group of the
        // warp's range, and that bookkeeping costs more than the idle rounds (measured: 13.3 against 11.7 us at 80 %).
        // (Two copies of the loop, so that the distance between two rows of a row group is a constant in each.)
        auto stream = [&](auto rgw_tag) {
            constexpr int RGW = decltype(rgw_tag)::value;  // positions between two rows of a row group: 4 or 1
            constexpr bool interleave = RGW > 1;
            const int rows_per = interleave ? (cnt + FC_WARPS - 1) / FC_WARPS : (cnt + NR - 1) / NR;
            int r_lo = min(cnt, (interleave ? warp : rg) * rows_per), r_hi = min(cnt, r_lo + rows_per);
            if constexpr (!interleave) {
                // Short lists are bound by latency, not by balance: an end of a range that lies within half a range of a
                // group boundary moves onto it, so that a row group mostly streams ONE group - all its row requests go
                // out together instead of one dependent batch per group.
                auto snap = [&](int b) {
                    int best = 0, dist = cnt + 1;
                    for (int g = 0; g <= ng; ++g) {
                        const int d = abs(s_goff[g] - b);
                        if (d < dist) { dist = d; best = s_goff[g]; }
                    }
                    return 2 * dist <= rows_per ? best : b;
                };
                r_lo = snap(min(cnt, rg * rows_per));
                r_hi = snap(min(cnt, (rg + 1) * rows_per));
            }
            const int jrg = interleave ? rg % (32 / LPR) : 0;
            int gl = 0;
            for (int t = r_lo; t < r_hi;) {
                while (gl + 1 < ng && s_goff[gl + 1] <= t) ++gl;   // group of list position t
                const int t_end = min(r_hi, s_goff[gl + 1]);
                const int p0 = t + ((jrg - (t - r_lo)) & (RGW - 1));  // this row group's first position of the stretch
                // the group's scales and zero points for this thread's columns (requested now, used below)
                const size_t gofs = (size_t)(g0 + gl) * N + col;
                const float4 *sp = reinterpret_cast<const float4 *>(qa.scale + gofs);
                const float4 s0 = __ldcg(sp), s1 = __ldcg(sp + 1), s2 = __ldcg(sp + 2), s3 = __ldcg(sp + 3);
                const uint4 zw = __ldcg(reinterpret_cast<const uint4 *>(qa.zero + gofs));
                unsigned long long acc2[BT][8];  // sum xv q of the stretch, 16 columns as 8 packed pairs
                float sx[BT];                    // sum xv of the stretch
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    sx[b] = 0.0f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc2[b][j] = 0ull;
                }
                // two register groups of U / 2 row loads alternate: one is used while the other is in flight
                constexpr int H = U / 2;
                uint2 va[H], vb[H];
                auto request = [&](uint2(&dst)[H], int first) {
#pragma unroll
                    for (int u = 0; u < H; ++u) {
                        const bool on = first + RGW * u < t_end;
                        dst[u] = ld_stream8_if(Wb + (size_t)(on ? s_k[first + RGW * u] : 0u) * row_bytes, on);
                    }
                };
                auto use = [&](const uint2(&src)[H], int first) {
#pragma unroll
                    for (int u = 0; u < H; ++u) {
                        if (first + RGW * u < t_end) {
#pragma unroll
                            for (int b = 0; b < BT; ++b) {
                                const float xv = s_xs[b * CAP + first + RGW * u];
                                sx[b] += xv;
                                fma_row_q4(acc2[b], src[u], xv);
                            }
                        }
                    }
                };
                request(va, p0);
                request(vb, p0 + RGW * H);
                for (int tb = p0; tb < t_end; tb += RGW * U) {
                    use(va, tb);
                    request(va, tb + RGW * U);
                    use(vb, tb + RGW * H);
                    request(vb, tb + RGW * (U + H));
                }
                // the stretch's contribution: scale (sum xv q - zero sum xv)
                const float sc[16] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w, s2.x, s2.y, s2.z, s2.w, s3.x, s3.y, s3.z, s3.w};
                const uint32_t z4[4] = {zw.x, zw.y, zw.z, zw.w};
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    float acc[16];
#pragma unroll
                    for (int j = 0; j < 8; ++j) unpack2(acc2[b][j], acc[2 * j], acc[2 * j + 1]);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float zf = (float)((z4[j >> 2] >> (8 * (j & 3))) & 255u);
                        y_acc[b][j] = fmaf(sc[j], fmaf(-zf, sx[b], acc[j]), y_acc[b][j]);
                    }
                }
                t = t_end;
            }
        };
        if (col_ok) {
            if (cnt >= NR * 24) stream(std::integral_constant<int, 32 / LPR>{});
            else stream(std::integral_constant<int, 1>{});
        }
        __syncthreads();
    }

    if (first_fill) prefetch_bias<true, EPI, TNT>(a, tile, s, per, bias0, bias1);  // a rank without groups
    // ---- reduction over the row groups (group order) and asynchronous cluster exchange, as in the 16-bit kernel: every
    // sum goes to the rank that owns its column as a store that counts down that rank's barrier; a rank finishes when
    // its own S partials are in.
    if (S > 1) cluster_wait();  // every rank's barrier is initialised (all ranks arrived at kernel start)
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
        float4 *dst = reinterpret_cast<float4 *>(s_red + ((rg * RB + rb) * TNT + cl * Q4_CPT));
#pragma unroll
        for (int q = 0; q < 4; ++q)
            dst[q] = make_float4(y_acc[rb][4 * q], y_acc[rb][4 * q + 1], y_acc[rb][4 * q + 2], y_acc[rb][4 * q + 3]);
    }
    __syncthreads();
    if (S > 1) {
        reduce_send_round<BT, EPI, TNT, NR, RB>(s_red, 0, B, s, per, smem_addr(s_gather), bar);
        bool landed = false;
        for (uint32_t it = 0; it < (1u << 22) && !landed; ++it) landed = mbarrier_try_wait(bar, 0);
        if (!landed && a.status) atomicCAS(a.status, 0, 2);  // never in a correct run; the result is then incomplete
    } else {
        float *owner[MAX_CLUSTER];
#pragma unroll
        for (int q = 0; q < MAX_CLUSTER; ++q) owner[q] = s_gather;
        reduce_push_round<BT, EPI, TNT, NR, RB>(s_red, 0, B, s, per, owner);
        __syncthreads();
    }
    finish_columns<true, BT, EPI, TNT>(a, tile, s, per, s_gather, bias0, bias1);
}

constexpr int q4_smem(int BT) { return q4_main_bytes(BT) + BT * GATHER_LD * 4 + FC_WARPS * 4 + (Q4_MAXG + 1) * 4 + 16; }

// Split-K factor: the most CTAs (column tiles x S) that are all resident, with at least one group per rank.
static int q4_split(int K, int N, int group) {
    const int tiles = (N + Q4_TN - 1) / Q4_TN, G = (K + group - 1) / group;
    int best_S = 1;
    long long best = -1;
    for (int S = 1; S <= MAX_CLUSTER; ++S) {
        if (g_tune.split_k > 0 && S > g_tune.split_k) continue;
        if (S > G) continue;
        const long long ctas = (long long)tiles * S;
        if (S > 1 && ctas > resident_ctas(S)) continue;
        if (ctas >= best) { best = ctas; best_S = S; }
    }
    return best_S;
}

template <int BT, int MODE, typename XT, int PUT>
static cudaError_t launch_q4_pu(const Q4Args &qa, cudaStream_t st) {
    static SmemOptIn opt_in;
    auto kern = fc_q4_kernel<BT, MODE, XT, PUT>;
    cudaError_t e0 = ensure_dynamic_smem(kern, q4_smem(BT), opt_in);
    if (e0 != cudaSuccess) return e0;
    return launch_cluster(kern, dim3((qa.f.ldw + Q4_TN - 1) / Q4_TN, qa.f.S), dim3(FC_THREADS), q4_smem(BT), qa.f.S, st, g_tune.pdl != 0, qa);
}

// 4, 6 or 8 chunk slots per warp: the fewest whose fill (slots x 256 channels) holds a whole group and, if possible,
// all groups of a rank.
template <int BT, int MODE, typename XT>
static cudaError_t launch_q4_t(const Q4Args &qa, cudaStream_t st) {
    const int group = qa.group, G = (qa.f.K + group - 1) / group, gper = (G + qa.f.S - 1) / qa.f.S;
    const int need = (gper * group / 32 + FC_WARPS - 1) / FC_WARPS;  // slots that take the rank's channels in one fill
    if (need <= 4 && group <= 4 * FC_WARPS * 32) return launch_q4_pu<BT, MODE, XT, 4>(qa, st);
    if (need <= 6 && group <= 6 * FC_WARPS * 32) return launch_q4_pu<BT, MODE, XT, 6>(qa, st);
    return launch_q4_pu<BT, MODE, XT, fc_pu(BT)>(qa, st);
}

// xkind: 0 fp16, 1 bf16, 2 float activations.  Batches beyond two rows run two rows at a time (row results are
// independent; the union mask then spans two rows).
static cudaError_t launch_q4(int mode, int xkind, Q4Args qa, cudaStream_t st) {
    const int B = qa.f.B;
    const size_t xsz = xkind == 2 ? 4 : 2;
    const unsigned char *x0 = static_cast<const unsigned char *>(qa.f.x);
    float *y0 = qa.f.y;
    for (int b0 = 0; b0 < B; b0 += 2) {
        qa.f.B = B - b0 >= 2 ? 2 : 1;
        qa.f.x = x0 + (size_t)b0 * qa.f.x_ld * xsz;
        qa.f.y = y0 + (size_t)b0 * qa.f.y_ld;
        cudaError_t e;
        if (qa.f.B == 1) {
            if (mode == MODE_DENSE) e = xkind == 2 ? launch_q4_t<1, MODE_DENSE, float>(qa, st) : xkind == 1 ? launch_q4_t<1, MODE_DENSE, __nv_bfloat16>(qa, st) : launch_q4_t<1, MODE_DENSE, __half>(qa, st);
            else e = xkind == 1 ? launch_q4_t<1, MODE_GATHER, __nv_bfloat16>(qa, st) : launch_q4_t<1, MODE_GATHER, __half>(qa, st);
        } else {
            if (mode == MODE_DENSE) e = xkind == 1 ? launch_q4_t<2, MODE_DENSE, __nv_bfloat16>(qa, st) : launch_q4_t<2, MODE_DENSE, __half>(qa, st);
            else e = xkind == 1 ? launch_q4_t<2, MODE_GATHER, __nv_bfloat16>(qa, st) : launch_q4_t<2, MODE_GATHER, __half>(qa, st);
        }
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace scap

using namespace scap;

extern "C" {

static scap_status q4_check(const void *x, const void *Wq, const float *scale, const unsigned char *zero, int group, const float *m,
                            const float *b, float *y, int B, int K, int N, scap_dtype xdt, const void *ws, size_t ws_bytes) {
    if (!x || !Wq || !scale || !zero || !y || !ws) return SCAP_ERR_INVALID_ARG;
    if (xdt != SCAP_F16 && xdt != SCAP_BF16) return SCAP_ERR_DTYPE;
    if (B < 1 || B > SCAP_MAX_BATCH || K < 1 || N < 1 || K > SCAP_MAX_K) return SCAP_ERR_SHAPE;
    if (group < 32 || group % 32 != 0 || group > 2048) return SCAP_ERR_SHAPE;
    if (N % 16 != 0 || !aligned16(x) || !aligned16(Wq) || !aligned16(scale) || !aligned16(zero) || !aligned16(y) || !aligned16(ws) ||
        (m && !aligned16(m)) || (b && !aligned16(b)))
        return SCAP_ERR_ALIGN;
    if (ws_bytes < scap_fc_workspace(B, K, N)) return SCAP_ERR_WORKSPACE;
    return check_device();
}

static void q4_fill(Q4Args &qa, const void *x, const void *Wq, const float *scale, const unsigned char *zero, int group, float *y, int B,
                    int K, int N) {
    memset(&qa, 0, sizeof(qa));
    qa.f.W = Wq; qa.f.K = K; qa.f.ldw = N; qa.f.Nh = N; qa.f.B = B; qa.f.tn = Q4_TN; qa.f.S = q4_split(K, N, group);
    qa.f.x = x; qa.f.x_ld = K; qa.f.y = y; qa.f.y_ld = N;
    qa.scale = scale; qa.zero = zero; qa.group = group;
    qa.f.status = tc_status_ptr();
}

scap_status scap_sparse_fc_q4(const void *x, scap_dtype xdt, const unsigned char *Wq, const float *scale, const unsigned char *zero,
                              int group, const float *m, const float *tau, const float *b_fused, float *y, int B, int K, int N,
                              uint32_t *idx_out, int *nnz_out, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!tau) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q4_check(x, Wq, scale, zero, group, m, b_fused, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    if ((idx_out || nnz_out) && B > 2) return SCAP_ERR_SHAPE;  // the kept list describes one launch (at most two rows)
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    Q4Args qa;
    q4_fill(qa, x, Wq, scale, zero, group, y, B, K, N);
    qa.f.m = m; qa.f.tau = tau; qa.f.bias = b_fused;
    const bool inspect = idx_out || nnz_out;
    if (inspect) qa.f.bits = reinterpret_cast<uint32_t *>(ws);
    cudaError_t e = launch_q4(MODE_GATHER, xdt == SCAP_BF16 ? 1 : 0, qa, st);
    if (e != cudaSuccess) return cuda_status(e);
    if (inspect) e = launch_expand_bits(qa.f.bits, K, idx_out, nnz_out, st);
    return cuda_status(e);
}

scap_status scap_dense_fc_q4(const void *x, scap_dtype xdt, const unsigned char *Wq, const float *scale, const unsigned char *zero,
                             int group, const float *b, float *y, int B, int K, int N, void *ws, size_t ws_bytes, scap_stream_t stream) {
    scap_status stt = q4_check(x, Wq, scale, zero, group, nullptr, b, y, B, K, N, xdt, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    Q4Args qa;
    q4_fill(qa, x, Wq, scale, zero, group, y, B, K, N);
    qa.f.bias = b;
    return cuda_status(launch_q4(MODE_DENSE, xdt == SCAP_BF16 ? 1 : 0, qa, reinterpret_cast<cudaStream_t>(stream)));
}

scap_status scap_fold_bias_q4(const unsigned char *Wq, const float *scale, const unsigned char *zero, int group, const float *m,
                              const float *b, int K, int N, float *b_fused, void *ws, size_t ws_bytes, scap_stream_t stream) {
    if (!m) return SCAP_ERR_INVALID_ARG;
    scap_status stt = q4_check(m, Wq, scale, zero, group, nullptr, b, b_fused, 1, K, N, SCAP_BF16, ws, ws_bytes);
    if (stt != SCAP_OK) return stt;
    Q4Args qa;
    q4_fill(qa, m, Wq, scale, zero, group, b_fused, 1, K, N);
    qa.f.bias = b;
    qa.f.hold_dependents = 1;  // it writes a parameter: ordinary stream order on both sides
    return cuda_status(launch_q4(MODE_DENSE, 2, qa, reinterpret_cast<cudaStream_t>(stream)));
}

}  // extern "C"
