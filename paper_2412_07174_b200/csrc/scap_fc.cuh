// The fused decode-time sparse FC kernel (Eq. 2-3, Eq. 6, Alg. 3).
//
// One kernel does centre + threshold + compaction + gather-GEMV + reduction:
//   grid  = (column tiles, S)   block = 256 threads
//   the S CTAs of a column tile form one thread-block cluster; CTA s owns the 32-channel chunks
//   c = s, s+S, s+2S, ... of the input, thresholds them itself (ballot + popcount, order kept),
//   streams the surviving weight rows of its tile with 16-byte loads kept U deep per thread, and
//   the cluster exchanges its S partial tiles through distributed shared memory and adds them in rank order.
// No global scratch, no atomics, no second kernel; the summation order is fixed, so results are
// bitwise reproducible.  Internal header shared by the FC, SwiGLU and MoE entry points.
#pragma once

#include <cooperative_groups.h>

#include "scap_common.cuh"

namespace scap {

namespace cg = cooperative_groups;

enum { MODE_GATHER = 0, MODE_DENSE = 1 };
enum { EPI_BIAS = 0, EPI_GLU = 1 };

constexpr int TN = 256;         // widest column tile per CTA (each thread owns 8 columns = one 16-byte load per row)
constexpr int MAX_CLUSTER = 8;  // portable cluster size: upper bound of the split-K factor S

constexpr int FC_THREADS = 256;  // 8 warps; two CTAs fit on an SM, so every cluster of the grid is resident at once
constexpr int FC_WARPS = FC_THREADS / 32;
__host__ __device__ constexpr int fc_min_blocks(int BT) { return 2; }
// chunks (of 32 channels) each warp thresholds per fill; their centred values stay in registers
__host__ __device__ constexpr int fc_pu(int BT) { return BT <= 2 ? 8 : BT <= 4 ? 6 : BT <= 8 ? 2 : 1; }
__host__ __device__ constexpr int fc_cap(int BT) { return FC_WARPS * fc_pu(BT) * 32; }  // channels staged per fill
__host__ __device__ constexpr int fc_rb(int BT) { return BT < 4 ? BT : 4; }              // batch rows per cross-warp round
__host__ __device__ constexpr int fc_unroll(int BT) { return BT <= 1 ? 16 : BT <= 4 ? 8 : 4; }  // row loads in flight per thread

__host__ __device__ constexpr int fc_main_bytes(int BT) {
    const int stage = fc_cap(BT) * 4 * (1 + BT);
    const int red = FC_WARPS * fc_rb(BT) * TN * 4;
    return stage > red ? stage : red;
}
// Row pitch of the gathered-partials region: a rank finishes ceil(columns / S) columns, so with a cluster size
// that does not divide the tile the S slices together are up to 2 * (S - 1) entries longer than the tile.
constexpr int GATHER_LD = TN + 16;
__host__ __device__ constexpr int fc_smem_bytes(int BT) {  // main | gathered partials | chunk masks | row map
    return fc_main_bytes(BT) + BT * GATHER_LD * 4 + (fc_cap(BT) / 32) * 4 + 16 * 4 + FC_WARPS * 4 + 16;
}

struct FcArgs {
    const void *W;        // [K, ldw] storage dtype, row k = all outputs of input channel k
    int K, ldw;           // ldw: columns of a weight row (N, or 2F for the packed gate|up weight)
    int Nh;               // EPI_BIAS: N.  EPI_GLU: F (gate columns 0..F-1, up columns F..2F-1)
    int B, S;             // batch rows; split-K factor = cluster size (1 .. 8)
    int tn;               // columns per CTA: 256 or 128
    const void *x;        // activations [rows, x_ld] of type XT
    int x_ld;
    const int *in_rows;   // batch row b reads row in_rows[b] of x (NULL: row b)
    const float *m;       // [K] or NULL
    const float *tau;     // [1] (MODE_GATHER)
    const float *bias;    // fp32 [ldw] or NULL
    const void *bias16;   // storage-dtype bias added on top (bias folding) or NULL
    float *y;             // EPI_BIAS: [rows, y_ld] ; EPI_GLU: z [rows, y_ld] (fp32)
    int y_ld;
    const int *out_rows;  // batch row b writes row out_rows[b] of y (NULL: row b)
    float *z_copy;        // EPI_GLU: optional second copy of z, [B, F] dense rows
    uint32_t *bits;       // optional [ceil(K/32)]: union keep mask, one word per 32-channel chunk
    int hold_dependents;  // 1: do not let the next kernel start before this grid completes (it writes parameters)
    int no_tc;            // 1: keep this call off the tcgen05 kernel
    int act;              // EPI_BIAS: 1 = the exact GELU is applied to the biased result (z_copy then gets a copy)
    const float *wscale;  // 8-bit weights only: one scale per input channel, W[k,n] = wscale[k] * Wq[k,n]
    int head_rows;        // fp32-FMA body: chunks per CTA whose rows are asked into L2 at kernel start (0: none)
    int l2_hints;         // fp32-FMA body: 1 = loads carry L2 eviction hints (keep x and m, stream W)
    int *status;          // device status word: set when a bounded wait runs out (NULL: not recorded)
    int spin;             // tcgen05 kernel: polls before a shared-memory barrier wait gives up (0: the built-in limit)
};

template <bool BF16, int BT, int CAP>
__device__ __forceinline__ void fma_row(float (&acc)[BT][8], const uint4 &v, const float *__restrict__ s_xs, int i) {
    float w[8];
    widen2<BF16>(v.x, w[0], w[1]);
    widen2<BF16>(v.y, w[2], w[3]);
    widen2<BF16>(v.z, w[4], w[5]);
    widen2<BF16>(v.w, w[6], w[7]);
#pragma unroll
    for (int b = 0; b < BT; ++b) {
        const float xv = s_xs[b * CAP + i];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[b][j] = fmaf(xv, w[j], acc[b][j]);
    }
}

// ---- 8-bit weights (WB = 1 in the body below): a 16-byte load holds 16 columns of a row.
// Two fp32 values in one 64-bit register, for the packed fp32 instructions of sm_100 (add.f32x2 / fma.rn.f32x2: one
// instruction per two weights).
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    return ((unsigned long long)__float_as_uint(hi) << 32) | (unsigned long long)__float_as_uint(lo);  // a register pair, no instruction
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
    lo = __uint_as_float((uint32_t)v);
    hi = __uint_as_float((uint32_t)(v >> 32));
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

// Exact GELU, gelu(v) = v/2 (1 + erf(v / sqrt 2)), binary32.
__device__ __forceinline__ float gelu_exact(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752f)); }

// Stores one finished EPI_BIAS result (activation applied first, if any).
__device__ __forceinline__ void store_result(const FcArgs &a, int row, int b, int n, float v) {
    if (a.act == 1) v = gelu_exact(v);
    a.y[(size_t)row * a.y_ld + n] = v;
    if (a.z_copy) a.z_copy[(size_t)b * a.Nh + n] = v;
}

template <bool BF16>
__device__ __forceinline__ float load_bias(const FcArgs &a, int n) {
    float bv = a.bias ? __ldcg(a.bias + n) : 0.0f;
    if (a.bias16) bv += widen_bits<BF16>(__ldcg(reinterpret_cast<const unsigned short *>(a.bias16) + n));
    return bv;
}

// One round of the reduction over NRED row groups (in group order) for RBX batch rows starting at b0: thread i
// sums column c of row rb from s_red[g][rb][c] and pushes the result into the shared memory of the cluster rank
// that owns the column (slot = this rank s).  EPI_GLU: owner by pair index j = c mod HALF; the gate and up
// values of a pair sit side by side in the owner's slot.
template <int BT, int EPI, int TNT, int NRED, int RBX>
__device__ __forceinline__ void reduce_push_round(const float *__restrict__ s_red, int b0, int B, int s, int per,
                                                  float *const (&owner)[MAX_CLUSTER]) {
    constexpr int HALF = TNT / 2;
    for (int i = threadIdx.x; i < RBX * TNT; i += FC_THREADS) {
        const int rb = i / TNT, c = i - rb * TNT, b = b0 + rb;
        float v = 0.0f;
#pragma unroll
        for (int g = 0; g < NRED; ++g) v += s_red[(g * RBX + rb) * TNT + c];
        if (b < B) {
            int r, slot;
            if constexpr (EPI == EPI_GLU) {
                const int j = c % HALF, hf = c / HALF;
                r = j / per;
                slot = ((s * BT + b) * 2 + hf) * per + (j - r * per);
            } else {
                r = c / per;
                slot = (s * BT + b) * per + (c - r * per);
            }
#pragma unroll
            for (int q = 0; q < MAX_CLUSTER; ++q)
                if (q == r) owner[q][slot] = v;
        }
    }
}

// The same reduction round with the asynchronous exchange: every element goes to its owner as a store that counts
// down the owner's shared-memory barrier when it lands.
template <int BT, int EPI, int TNT, int NRED, int RBX>
__device__ __forceinline__ void reduce_send_round(const float *__restrict__ s_red, int b0, int B, int s, int per, uint32_t gather_local,
                                                  uint32_t bar_local) {
    constexpr int HALF = TNT / 2;
    for (int i = threadIdx.x; i < RBX * TNT; i += FC_THREADS) {
        const int rb = i / TNT, c = i - rb * TNT, b = b0 + rb;
        float v = 0.0f;
#pragma unroll
        for (int g = 0; g < NRED; ++g) v += s_red[(g * RBX + rb) * TNT + c];
        if (b < B) {
            int r, slot;
            if constexpr (EPI == EPI_GLU) {
                const int j = c % HALF, hf = c / HALF;
                r = j / per;
                slot = ((s * BT + b) * 2 + hf) * per + (j - r * per);
            } else {
                r = c / per;
                slot = (s * BT + b) * per + (c - r * per);
            }
            st_async_f32(cluster_addr(gather_local + 4u * (uint32_t)slot, (uint32_t)r), v, cluster_addr(bar_local, (uint32_t)r));
        }
    }
}

// After the cluster barrier: every rank adds the S partials of its columns in rank order, adds the bias (or forms
// z = up * silu(gate)) and writes the result.
template <bool BF16, int BT, int EPI, int TNT>
__device__ __forceinline__ void finish_columns(const FcArgs &a, int tile, int s, int per, const float *__restrict__ s_gather,
                                               const float (&bias0)[2], const float (&bias1)[2]) {
    constexpr int HALF = TNT / 2;
    const int B = a.B, S = a.S, tid = threadIdx.x;
    for (int it = 0; tid + it * FC_THREADS < per * B; ++it) {
        const int i = tid + it * FC_THREADS;
        const int b = i / per, c = i - b * per;
        const int row = a.out_rows ? __ldcg(a.out_rows + b) : b;
        if constexpr (EPI == EPI_BIAS) {
            const int n = tile * TNT + s * per + c;
            if (s * per + c < TNT && n < a.Nh) {
                float v = it == 0 ? bias0[0] : it == 1 ? bias0[1] : load_bias<BF16>(a, n);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) v += s_gather[(q * BT + b) * per + c];
                store_result(a, row, b, n, v);
            }
        } else {
            const int F = a.Nh, f = tile * HALF + s * per + c;
            if (s * per + c < HALF && f < F) {
                float g = it == 0 ? bias0[0] : it == 1 ? bias0[1] : (a.bias ? __ldcg(a.bias + f) : 0.0f);
                float u = it == 0 ? bias1[0] : it == 1 ? bias1[1] : (a.bias ? __ldcg(a.bias + F + f) : 0.0f);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) {
                        g += s_gather[((q * BT + b) * 2 + 0) * per + c];
                        u += s_gather[((q * BT + b) * 2 + 1) * per + c];
                    }
                const float z = u * (g / (1.0f + expf(-g)));  // up * silu(gate)
                a.y[(size_t)row * a.y_ld + f] = z;
                if (a.z_copy) a.z_copy[(size_t)b * F + f] = z;
            }
        }
    }
}

// Bias of the columns this rank finishes, requested (through L2) before the row stream starts so that the load is off
// the critical path.
template <bool BF16, int EPI, int TNT>
__device__ __forceinline__ void prefetch_bias(const FcArgs &a, int tile, int s, int per, float (&bias0)[2], float (&bias1)[2]) {
    constexpr int HALF = TNT / 2;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        bias0[it] = bias1[it] = 0.0f;
        const int i = threadIdx.x + it * FC_THREADS;
        if (i < per * a.B) {
            const int c = i % per;
            if constexpr (EPI == EPI_GLU) {
                const int f = tile * HALF + s * per + c;
                if (s * per + c < HALF && f < a.Nh && a.bias) { bias0[it] = __ldcg(a.bias + f); bias1[it] = __ldcg(a.bias + a.Nh + f); }
            } else {
                const int n = tile * TNT + s * per + c;
                if (s * per + c < TNT && n < a.Nh) bias0[it] = load_bias<BF16>(a, n);
            }
        }
    }
}

// Body for column tile `tile` and cluster rank `s`; every thread of every CTA of the cluster calls it.
// TNT = columns per CTA (256 or 128): a row segment is TNT/8 lanes wide, so a warp streams 1 or 2 rows per load.
// With wait_inside the body itself waits for the previous kernel in the stream before it reads anything: the
// activations, and equally tau, m and the biases, may have been written by any earlier work on the stream.  No load
// or prefetch goes out before that wait (measured: memory operations issued ahead of it delay its return for the
// CTAs that become resident late, 0.15 - 0.2 us per call), and everything a kernel may rewrite is read through L2.
// PUT = chunk slots per warp and fill that the threshold code is unrolled for (at most fc_pu(BT), which sizes the
// shared-memory list): that code is bound by instruction issue, so the launcher picks the smallest instantiation
// that still takes the rank's channels in one fill.
// WB = bytes per weight: 2 (fp16 / bf16) or 1 (signed 8-bit with one binary32 scale per input channel, which is folded
// into the pruned activation once per kept channel, so the stream multiplies by the raw integers).  A thread's 16-byte
// load then covers 16 columns and 8 lanes cover a row of a 128-column tile.
template <bool BF16, int BT, int MODE, typename XT, int EPI, int TNT, int PUT = fc_pu(BT), int WB = 2>
__device__ __forceinline__ void fc_body(const FcArgs &a, const int tile, const int s, const bool wait_inside) {
    constexpr int NT = FC_THREADS, PU = PUT, CAP = fc_cap(BT), RB = fc_rb(BT), U = fc_unroll(BT);
    constexpr int CAPC = FC_WARPS * PU;  // chunks per fill
    static_assert(PUT >= 1 && PUT <= fc_pu(BT), "the list is sized for fc_pu(BT) slots per warp");
    static_assert(WB == 2 || (WB == 1 && EPI == EPI_BIAS && TNT == 128), "8-bit weights: plain FC, 128-column tiles");
    constexpr int CPT = 16 / WB;      // columns per thread (one 16-byte load)
    constexpr int LPR = TNT / CPT;    // lanes per row segment
    constexpr int NR = NT / LPR;      // row groups per CTA: group g streams rows g, g+NR, ...
    constexpr int HALF = TNT / 2;
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *s_k = reinterpret_cast<uint32_t *>(smem);
    float *s_xs = reinterpret_cast<float *>(smem) + CAP;
    float *s_red = reinterpret_cast<float *>(smem);
    float *s_gather = reinterpret_cast<float *>(smem + fc_main_bytes(BT));  // [S][BT][columns owned by this rank]
    uint32_t *s_bits = reinterpret_cast<uint32_t *>(s_gather + BT * GATHER_LD);
    int *s_rows = reinterpret_cast<int *>(s_bits + CAPC);  // source row of x per batch row (when a row map is given)
    int *s_wcnt = s_rows + 16;                             // kept channels per warp, this fill
    const uint32_t bar = smem_addr(s_wcnt + FC_WARPS);     // 8 bytes: barrier the split-K partials of this rank's columns land on

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = tid / LPR, cl = tid % LPR;  // row group and column lane of this thread
    const int B = a.B, S = a.S, K = a.K;
    const XT *xg = reinterpret_cast<const XT *>(a.x);

    // this thread's 8 columns
    int col;
    bool col_ok;
    if constexpr (EPI == EPI_GLU) {  // first half of the column lanes: gate columns; second half: the matching up columns
        const int f = tile * HALF + (cl % (LPR / 2)) * 8;
        col_ok = f < a.Nh;
        col = (cl / (LPR / 2)) * a.Nh + f;
    } else {
        col = tile * TNT + cl * CPT;
        col_ok = col < a.Nh;
    }
    const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (size_t)col * WB;
    const size_t row_bytes = (size_t)a.ldw * WB;

    // Head of the stream, asked into L2 before anything is known about the activations: between the end of the
    // previous call and the first row request of this one (hand-over, activations and parameters through L2, compaction:
    // about 2 us) the memory system would otherwise idle.  The rows of the rank's first head_rows chunks are requested
    // as L2 hints - all of them, kept or not, so the part that is pruned is extra traffic, bought with idle time -
    // and the row requests proper then meet them in L2.  The weights are constants of the layer, so this precedes
    // the wait for earlier work on the stream.  One 128-byte line per hint: the lanes that start a line issue them.
    if (a.head_rows > 0 && col_ok && (cl & 7) == 0) {
        const int nhead = min(a.head_rows, (((K + 31) >> 5) - s + S - 1) / S) * 32;
        for (int t = rg; t < nhead; t += NR) {
            const int k = (s + S * (t >> 5)) * 32 + (t & 31);
            if (k < K) prefetch_l2(Wb + (size_t)k * row_bytes);
        }
    }

    // columns (EPI_GLU: gate/up pairs) this rank finishes after the cluster exchange
    const int per = ((EPI == EPI_GLU ? HALF : TNT) + S - 1) / S;  // the last rank may own fewer
    if (S > 1) {
        // This rank will receive S * B * (columns it owns) partial sums (gate and up: twice that) on its barrier.
        // The fence after the initialisation publishes the barrier; the arrival half of a cluster barrier follows (with
        // no ordering of its own, so it waits for nothing: the releasing form took 0.3 - 0.8 us, measured, on the
        // critical path of a CTA that became resident late) and the waiting half sits before the first send, by which
        // time every rank has long arrived.
        if (tid == 0) {
            const int owned = max(0, min(per, (EPI == EPI_GLU ? HALF : TNT) - s * per));
            mbarrier_init(bar, 1);
            mbarrier_arrive_expect(bar, (uint32_t)(S * B * owned * (EPI == EPI_GLU ? 8 : 4)));
        }
        cluster_arrive_relaxed();
    }
    float bias0[2], bias1[2];

    float acc[BT][CPT];
    unsigned long long acc2[BT][8];  // WB = 1: 16 columns per batch row as 8 packed pairs
#pragma unroll
    for (int b = 0; b < BT; ++b) {
#pragma unroll
        for (int j = 0; j < CPT; ++j) acc[b][j] = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) acc2[b][j] = 0ull;
    }

    const int nchunks = (K + 31) >> 5;
    const int my_chunks = nchunks > s ? (nchunks - s + S - 1) / S : 0;  // chunks s, s+S, ...
    float tau = 0.0f;
    // x and m are read again by every column tile of the call (and m by every later call): ask L2 to keep them and
    // to drop the weight rows, which are read once, first.
    const uint64_t pol_keep = a.l2_hints ? l2_policy_keep() : l2_policy_normal();
    const uint64_t pol_stream = a.l2_hints ? l2_policy_stream() : l2_policy_normal();

    // The wait for the previous kernel sits behind the address arithmetic of the first fill (pure register work, which
    // so overlaps the previous kernel's tail); with a row map, or without channels, it comes first.
    bool waited = !wait_inside;
    if (!waited && (a.in_rows || my_chunks == 0)) {
        griddep_wait();
        griddep_launch_dependents();
        waited = true;
    }
    if (a.in_rows) {  // one L2 read per CTA and row (the map is an output of the previous kernel), then broadcast
        if (tid < BT) s_rows[tid] = __ldcg(a.in_rows + (tid < B ? tid : 0));
        __syncthreads();
    }
    // tau: one request per CTA (thousands of simultaneous requests for one address queue up in its L2 slice), issued
    // first and handed to the other warps through shared memory once the loads of the first fill are in flight
    float tau_reg = 0.0f;
    bool bias_done = false;
    const int kstep = S * 32;  // channel distance between consecutive chunks of a rank
    for (int j0 = 0; j0 < my_chunks; j0 += CAPC) {
        const int nj = min(CAPC, my_chunks - j0);
        const int pw = (nj + FC_WARPS - 1) / FC_WARPS;  // chunks per warp this fill: warp w owns chunks w * pw .. w * pw + pw - 1
        // ---- A: every warp loads its chunks at once, centres and thresholds them (Alg. 3: one binary32 subtraction, one
        // compare per element) and keeps the values in registers.  This code runs once per fill on all sixteen warps
        // of the SM at the same moment, so it is bound by instruction issue: a slot costs one address add, one
        // compare and the predicated load (unused slots are predicated off, no branch), and nothing consumes a value
        // inside the load loops, so the loads of a lane are all in flight together.
        const int nw = max(0, min(pw, nj - warp * pw));         // chunks of this warp
        const int kbase = (s + S * (j0 + warp * pw)) * 32 + lane;  // this lane's channel in the warp's first chunk
        const XT *xrow[BT];
#pragma unroll
        for (int b = 0; b < BT; ++b) xrow[b] = xg + (size_t)(a.in_rows ? s_rows[b < B ? b : 0] : (b < B ? b : 0)) * a.x_ld + kbase;
        const float *mrow = a.m ? a.m + kbase : nullptr;
        bool okx[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) okx[p] = p < nw && kbase + p * kstep < K;
        if (!waited) {
            griddep_wait();               // everything earlier work on the stream wrote (activations, parameters) is complete and visible
            griddep_launch_dependents();  // the next kernel may begin launching; it waits for this grid itself
            waited = true;
        }
        if (MODE == MODE_GATHER && j0 == 0 && tid == 0) tau_reg = ld_act(a.tau);
        XT xraw[PU][BT];
        float xv[PU][BT], mk[PU];
        // (Skipping the unused slots of a fill with CTA-uniform branches was measured: 0.9 us per call slower - the
        // branches break up the batch of loads.)
#pragma unroll
        for (int p = 0; p < PU; ++p) {
#pragma unroll
            for (int b = 0; b < BT; ++b) xraw[p][b] = ld_act_if(xrow[b] + p * kstep, okx[p] && b < B, pol_keep);
        }
#pragma unroll
        for (int p = 0; p < PU; ++p) mk[p] = ld_act_if(mrow + p * kstep, mrow != nullptr && okx[p], pol_keep);
        float sc[WB == 1 ? PU : 1];
        if constexpr (WB == 1) {
#pragma unroll
            for (int p = 0; p < PU; ++p) sc[p] = ld_act_if(a.wscale + kbase + p * kstep, okx[p], pol_keep);
        }
        if (MODE == MODE_GATHER && j0 == 0) {
            float *s_tau = reinterpret_cast<float *>(s_wcnt + FC_WARPS + 2);  // behind the 8-byte barrier
            if (tid == 0) *s_tau = tau_reg;
            __syncthreads();
            tau = *s_tau;
        }
#pragma unroll
        for (int p = 0; p < PU; ++p)
#pragma unroll
            for (int b = 0; b < BT; ++b) xv[p][b] = widen1(xraw[p][b]);
        // Branch-free so that the PU independent chains interleave: keep masks, then one ballot word per chunk.
        uint32_t km[PU];
        unsigned bal[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const bool ok = okx[p];
            uint32_t m_ = 0;
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                if constexpr (MODE == MODE_GATHER) {
                    const float dv = a.m ? __fsub_rn(xv[p][b], mk[p]) : xv[p][b];
                    xv[p][b] = dv;
                    m_ |= (ok && b < B && fabsf(dv) >= tau) ? (1u << b) : 0u;
                } else {
                    m_ = ok ? 1u : 0u;  // dense: every channel, no compare
                }
            }
            km[p] = m_;
            bal[p] = __ballot_sync(0xffffffffu, m_ != 0);
        }
        // ---- position of each chunk in the kept list.  A warp owns PU consecutive chunks, so the positions inside
        // the warp's stretch follow from its own ballot words; only the eight per-warp totals cross warps.
        int my_off[PU], wtotal = 0;
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            my_off[p] = wtotal;
            wtotal += __popc(bal[p]);
        }
        if (lane == 0) s_wcnt[warp] = wtotal;
        if (MODE == MODE_GATHER && a.bits && tile == 0) {  // lane p publishes the mask word of the warp's p-th chunk
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
        // ---- B: kept channels and their pruned values, in ascending channel order
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            if (km[p]) {
                const int pos = wbase + my_off[p] + __popc(bal[p] & ((1u << lane) - 1u));
                s_k[pos] = (uint32_t)(kbase + p * kstep);
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    float v = (MODE == MODE_DENSE || ((km[p] >> b) & 1u)) ? xv[p][b] : 0.0f;
                    if constexpr (WB == 1) v = __fmul_rn(v, sc[p]);  // the channel's weight scale, once per kept channel
                    s_xs[b * CAP + pos] = v;
                }
            }
        }
        __syncthreads();

        // ---- stream the kept rows: row group g takes rows g, g+NR, ...  Two register groups of G loads alternate
        // (one is consumed while the other is in flight).
        if (col_ok) {
            constexpr int G = U / 2;
            const int nrows = cnt > rg ? (cnt - rg + NR - 1) / NR : 0;
            uint4 ga[G], gb[G];
            // the first 2 G requests go out without a branch (predicated loads; list entries beyond the count are
            // never dereferenced)
#pragma unroll
            for (int u = 0; u < G; ++u)
                ga[u] = ld_stream16_if(Wb + (size_t)s_k[rg + NR * u] * row_bytes, u < nrows, pol_stream);
#pragma unroll
            for (int u = 0; u < G; ++u)
                gb[u] = ld_stream16_if(Wb + (size_t)s_k[rg + NR * (G + u)] * row_bytes, G + u < nrows, pol_stream);
            if (!bias_done) {  // behind the first row requests: needed only when the columns are finished
                prefetch_bias<BF16, EPI, TNT>(a, tile, s, per, bias0, bias1);
                bias_done = true;
            }
            auto use = [&](const uint4 &v, int t) {
                if constexpr (WB == 2) fma_row<BF16, BT, CAP>(acc, v, s_xs, rg + NR * t);
                else fma_row_q8<BT, CAP>(acc2, v, s_xs, rg + NR * t);
            };
            // Full rounds first: while every row of this round and of the next exists the body carries no compares and
            // no branches (they cost about as many instructions as the arithmetic of a row at batch 1); the guarded form
            // finishes the list.
            // (At batch 1 the second copy of the body costs more than it saves - measured, +0.2 us per sparse call on
            // either weight format - so only the instantiations for two and more rows take the full rounds:
            // -1.0 .. -1.7 us per call at batch 2 and 4, -2 .. -3 us at batch 2 on 8-bit weights.)
            constexpr bool FULL_ROUNDS = BT >= 2 || (WB == 1 && MODE == MODE_DENSE);  // (the dense 8-bit call gains 0.1 us)
            int t0 = 0;
            for (; FULL_ROUNDS && t0 + 4 * G <= nrows; t0 += 2 * G) {
#pragma unroll
                for (int u = 0; u < G; ++u) use(ga[u], t0 + u);
#pragma unroll
                for (int u = 0; u < G; ++u) ga[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 2 * G + u)] * row_bytes, pol_stream);
#pragma unroll
                for (int u = 0; u < G; ++u) use(gb[u], t0 + G + u);
#pragma unroll
                for (int u = 0; u < G; ++u) gb[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 3 * G + u)] * row_bytes, pol_stream);
            }
            for (; t0 < nrows; t0 += 2 * G) {
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + u < nrows) use(ga[u], t0 + u);
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + 2 * G + u < nrows) ga[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 2 * G + u)] * row_bytes, pol_stream);
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + G + u < nrows) use(gb[u], t0 + G + u);
#pragma unroll
                for (int u = 0; u < G; ++u)
                    if (t0 + 3 * G + u < nrows) gb[u] = ld_stream16(Wb + (size_t)s_k[rg + NR * (t0 + 3 * G + u)] * row_bytes, pol_stream);
            }
        }
        __syncthreads();
    }

    if (!bias_done) prefetch_bias<BF16, EPI, TNT>(a, tile, s, per, bias0, bias1);
    // ---- reduction over the row groups in group order; each finished element of this CTA's partial tile is
    // sent to the shared memory of the cluster rank that owns its column (slot = this rank) as an asynchronous
    // store that counts down the owner's barrier.  A rank finishes its columns as soon as its own S partials are
    // in - it neither waits for the other ranks' exchanges nor for an acknowledgement of its own stores - and adds
    // them in rank order.
    static_assert(RB == BT, "one reduction round");
    if (S > 1) cluster_wait();  // every rank's barrier is initialised (all ranks arrived at kernel start)
    // WB = 1: the four row groups of a warp (lanes l, l ^ 8, l ^ 16, l ^ 24 hold the same columns) are added by shuffles
    // in a fixed order first, so that the cross-warp reduction sees one partial per warp.
    constexpr int NRED = WB == 1 ? FC_WARPS : NR;
    if constexpr (WB == 1) {
#pragma unroll
        for (int b = 0; b < BT; ++b) {
#pragma unroll
            for (int j = 0; j < 8; ++j) unpack2(acc2[b][j], acc[b][2 * j], acc[b][2 * j + 1]);
#pragma unroll
            for (int j = 0; j < CPT; ++j) {
                acc[b][j] += __shfl_xor_sync(0xffffffffu, acc[b][j], 8);
                acc[b][j] += __shfl_xor_sync(0xffffffffu, acc[b][j], 16);
            }
        }
    }
    if (WB == 2 || lane < LPR) {
        const int g = WB == 1 ? warp : rg;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
            float4 *dst = reinterpret_cast<float4 *>(s_red + ((g * RB + rb) * TNT + cl * CPT));
#pragma unroll
            for (int q = 0; q < CPT / 4; ++q)
                dst[q] = make_float4(acc[rb][4 * q], acc[rb][4 * q + 1], acc[rb][4 * q + 2], acc[rb][4 * q + 3]);
        }
    }
    __syncthreads();
    if (S > 1) {
        reduce_send_round<BT, EPI, TNT, NRED, RB>(s_red, 0, B, s, per, smem_addr(s_gather), bar);
        bool landed = false;
        for (uint32_t it = 0; it < (1u << 22) && !landed; ++it) landed = mbarrier_try_wait(bar, 0);
        if (!landed && a.status) atomicCAS(a.status, 0, 2);  // never in a correct run; the result is then incomplete
    } else {
        float *owner[MAX_CLUSTER];
#pragma unroll
        for (int q = 0; q < MAX_CLUSTER; ++q) owner[q] = s_gather;
        reduce_push_round<BT, EPI, TNT, NRED, RB>(s_red, 0, B, s, per, owner);
        __syncthreads();
    }

    finish_columns<BF16, BT, EPI, TNT>(a, tile, s, per, s_gather, bias0, bias1);
}

// ------------------------------------------------------------------------------------------------
// Batch 3..16: the same kernel with the multiply-accumulate on the tensor cores.
//
// At more than two batch rows the fp32 FMA path issues 8 * B instructions per 16-byte weight load and the
// SM's issue rate, not HBM, becomes the limit.  Here a warp owns a 64-column chunk of the tile and streams
// blocks of 16 kept rows through mma.m16n8k16 (bf16 or fp16 operands, fp32 accumulation):
//   - lane (g, t) = (lane / 4, lane % 4) loads rows 2t, 2t+1, 2t+8, 2t+9 of the block at columns 8g .. 8g+7 of
//     the chunk; a byte permute pairs the two rows of each column, which is exactly the B fragment (k16 x n8)
//     of eight MMAs - MMA number i takes column i of every lane's eight, i.e. the column set {8g' + i};
//   - the A fragment (16 batch rows x 16 kept channels) comes from the staged activations.  They are fp32 values
//     (x - m), so each is split into NSPLIT parts of the weight dtype (bf16: hi + mid + lo = 24 mantissa bits,
//     fp16: hi + lo = 22 bits) and the tile is multiplied once per part: nothing is lost against the fp32 path.
//     (fp16 parts overflow for |x - m| > 65504.)
// ------------------------------------------------------------------------------------------------
// Two instantiations: ROWS = 8 (batch 3..8; the upper half of the 16-row tile is fed zeros and twice as many
// channels fit per fill) and ROWS = 16 (batch 9..16).  The template parameter BT of the kernels carries ROWS.
__host__ __device__ constexpr bool is_mma(int BT) { return BT == 8 || BT == 16; }
__host__ __device__ constexpr int mma_pu(int ROWS) { return ROWS == 8 ? 6 : 3; }              // chunks per warp per fill
__host__ __device__ constexpr int mma_cap(int ROWS) { return FC_WARPS * mma_pu(ROWS) * 32; }  // 1536 / 768 channels per fill
__host__ __device__ constexpr int mma_xld2(int ROWS) { return mma_cap(ROWS) / 2 + 4; }  // words per batch row of one staged part
__host__ __device__ constexpr int mma_nsplit(bool bf16) { return bf16 ? 3 : 2; }
__host__ __device__ constexpr int mma_main_bytes(int ROWS) {
    const int stage = mma_cap(ROWS) * 4 + 3 * ROWS * mma_xld2(ROWS) * 4;
    const int red = FC_WARPS * 64 * ROWS * 4;  // (8 / NCW) row groups x ROWS x (64 NCW) columns
    return stage > red ? stage : red;
}
__host__ __device__ constexpr int mma_smem_bytes(int ROWS) {
    return mma_main_bytes(ROWS) + ROWS * GATHER_LD * 4 + (mma_cap(ROWS) / 32) * 4 + 16 * 4 + 16;
}
__host__ __device__ constexpr int fc_smem_for(int BT) { return is_mma(BT) ? mma_smem_bytes(BT) : fc_smem_bytes(BT); }

template <bool BF16>
__device__ __forceinline__ void mma_k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if constexpr (BF16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Splits v into NSPLIT values of the weight dtype whose sum is v (bf16: exactly, unless a part falls below the
// binary32 normal range; fp16: to 2^-22); part[0] is the leading one.
template <bool BF16>
__device__ __forceinline__ void split_parts(float v, unsigned short (&part)[3]) {
    if constexpr (BF16) {
        // Truncation cuts the 24-bit significand into three consecutive 8-bit fields: hi = the upper half of the
        // pattern, r1 = v - hi (exact), mid = the upper half of r1, lo = r1 - mid (exact, at most 8 bits: a bf16).
        const uint32_t hb = __float_as_uint(v) & 0xffff0000u;
        const float r1 = v - __uint_as_float(hb);
        const uint32_t mb = __float_as_uint(r1) & 0xffff0000u;
        const float r2 = r1 - __uint_as_float(mb);
        part[0] = (unsigned short)(hb >> 16);
        part[1] = (unsigned short)(mb >> 16);
        part[2] = (unsigned short)(__float_as_uint(r2) >> 16);
    } else {
        const __half h = __float2half_rn(v);
        const __half l = __float2half_rn(v - __half2float(h));
        part[0] = __half_as_ushort(h);
        part[1] = __half_as_ushort(l);
        part[2] = 0;
    }
}

template <bool BF16, int ROWS, int MODE, typename XT, int EPI, int TNT>
__device__ __forceinline__ void fc_body_mma(const FcArgs &a, const int tile, const int s, const bool wait_inside) {
    constexpr int BT = ROWS, PU = mma_pu(ROWS), CAP = mma_cap(ROWS), XLD2 = mma_xld2(ROWS), CAPC = CAP / 32;
    constexpr int NSPLIT = mma_nsplit(BF16);
    constexpr int NCW = TNT / 64;          // warps across the columns of the tile
    constexpr int NRW = FC_WARPS / NCW;    // warps across row blocks: warp row rw streams blocks rw, rw+NRW, ...
    constexpr int HALF = TNT / 2;
    constexpr int G = 1;                   // row blocks per register group (two groups alternate); 4 loads per lane each
    extern __shared__ __align__(16) unsigned char smem[];
    uint32_t *s_k = reinterpret_cast<uint32_t *>(smem);
    uint32_t *s_xp = reinterpret_cast<uint32_t *>(smem) + CAP;                 // [NSPLIT][16][XLD2] packed pairs
    unsigned short *s_xh = reinterpret_cast<unsigned short *>(s_xp);           // same, addressed per element
    float *s_red = reinterpret_cast<float *>(smem);                            // [NRW][16][TNT]
    float *s_gather = reinterpret_cast<float *>(smem + mma_main_bytes(ROWS));
    uint32_t *s_bits = reinterpret_cast<uint32_t *>(s_gather + BT * GATHER_LD);
    int *s_rows = reinterpret_cast<int *>(s_bits + CAPC);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3, cw = warp % NCW, rw = warp / NCW;
    const int B = a.B, S = a.S, K = a.K;
    const XT *xg = reinterpret_cast<const XT *>(a.x);

    // this lane's 8 columns inside its warp's 64-column chunk
    int col;
    bool col_ok;
    if constexpr (EPI == EPI_GLU) {  // first half of the chunks: gate columns; second half: the matching up columns
        const int f = tile * HALF + (cw % (NCW / 2)) * 64 + g * 8;
        col_ok = f < a.Nh;
        col = (cw / (NCW / 2)) * a.Nh + f;
    } else {
        col = tile * TNT + cw * 64 + g * 8;
        col_ok = col < a.Nh;
    }
    const unsigned char *Wb = reinterpret_cast<const unsigned char *>(a.W) + (size_t)col * 2;
    const size_t row_bytes = (size_t)a.ldw * 2;

    const int per = ((EPI == EPI_GLU ? HALF : TNT) + S - 1) / S;  // the last rank may own fewer
    float bias0[2], bias1[2];

    float acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    const int nchunks = (K + 31) >> 5;
    const int my_chunks = nchunks > s ? (nchunks - s + S - 1) / S : 0;
    float tau = 0.0f;

    if (wait_inside) {  // nothing is read before earlier work on the stream is complete
        griddep_wait();
        griddep_launch_dependents();
    }
    if constexpr (MODE == MODE_GATHER) {
        float tv = 0.0f;
        if (lane == 0) tv = ld_act(a.tau);
        tau = __shfl_sync(0xffffffffu, tv, 0);
    }
    prefetch_bias<BF16, EPI, TNT>(a, tile, s, per, bias0, bias1);
    if (a.in_rows) {  // one L2 read per CTA and row, then broadcast
        if (tid < BT) s_rows[tid] = __ldcg(a.in_rows + (tid < B ? tid : 0));
        __syncthreads();
    }
    int rows_of[BT];  // source row of x for every batch row (clamped for the unused ones)
#pragma unroll
    for (int b = 0; b < BT; ++b) rows_of[b] = a.in_rows ? s_rows[b] : (b < B ? b : 0);

    const int Bp = (B + 3) & ~3;  // batch rows staged (groups of 4); fragment rows beyond them are fed zeros

    for (int j0 = 0; j0 < my_chunks; j0 += CAPC) {
        const int nj = min(CAPC, my_chunks - j0);
        // ---- A: keep masks.  Each warp takes PU chunks; all 16 * PU activation loads of a lane are in flight
        // together; the values are not kept (they are re-read in pass B) to stay within the registers.
        float mk[PU];
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = p * FC_WARPS + warp;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            mk[p] = a.m ? ld_act_if(a.m + k, j < nj && k < K) : 0.0f;
        }
        uint32_t km[PU];
        unsigned bal[PU];
        XT xraw[PU][BT];  // stays in registers until pass B
        {
#pragma unroll
            for (int p = 0; p < PU; ++p) {
                const int j = p * FC_WARPS + warp;
                const int k = (s + S * (j0 + j)) * 32 + lane;
                const bool ok = j < nj && k < K;
#pragma unroll
                for (int b = 0; b < BT; ++b) xraw[p][b] = ld_act_if(xg + (size_t)rows_of[b] * a.x_ld + k, ok && b < B);
            }
#pragma unroll
            for (int p = 0; p < PU; ++p) {
                const int j = p * FC_WARPS + warp;
                const int k = (s + S * (j0 + j)) * 32 + lane;
                const bool ok = j < nj && k < K;
                uint32_t m_ = 0;
                if constexpr (MODE == MODE_GATHER) {
#pragma unroll
                    for (int b = 0; b < BT; ++b) {
                        const float xv = widen1(xraw[p][b]);
                        const float dv = a.m ? __fsub_rn(xv, mk[p]) : xv;
                        m_ |= (ok && b < B && fabsf(dv) >= tau) ? (1u << b) : 0u;
                    }
                } else {
                    m_ = ok ? 1u : 0u;
                }
                km[p] = m_;
                bal[p] = __ballot_sync(0xffffffffu, m_ != 0);
            }
        }
        {
            unsigned mine = 0;
#pragma unroll
            for (int p = 0; p < PU; ++p) mine = lane == p ? bal[p] : mine;
            const int j = lane * FC_WARPS + warp;
            if (lane < PU && j < nj) {
                s_bits[j] = mine;
                if (MODE == MODE_GATHER && a.bits && tile == 0) a.bits[s + S * (j0 + j)] = mine;
            }
        }
        __syncthreads();
        int my_off[PU], cnt;
        {
            int c_lo[(CAPC + 31) / 32];
            cnt = 0;
#pragma unroll
            for (int q = 0; q < (CAPC + 31) / 32; ++q) {
                c_lo[q] = (q * 32 + lane < nj) ? __popc(s_bits[q * 32 + lane]) : 0;
                cnt += __reduce_add_sync(0xffffffffu, c_lo[q]);
            }
#pragma unroll
            for (int p = 0; p < PU; ++p) {
                int o = 0;
#pragma unroll
                for (int q = 0; q < (CAPC + 31) / 32; ++q)
                    o += __reduce_add_sync(0xffffffffu, (q * 32 + lane < p * FC_WARPS + warp) ? c_lo[q] : 0);
                my_off[p] = o;
            }
        }
        // ---- B: kept channels and the parts of their pruned values (same arithmetic as in A, from the same registers)
#pragma unroll
        for (int p = 0; p < PU; ++p) {
            const int j = p * FC_WARPS + warp;
            const int k = (s + S * (j0 + j)) * 32 + lane;
            const int pos = my_off[p] + __popc(bal[p] & ((1u << lane) - 1u));
            if (km[p]) {
                s_k[pos] = (uint32_t)k;
#pragma unroll
                for (int b = 0; b < BT; ++b) {
                    if (b < Bp) {  // rows beyond Bp are never read
                        const float xv = widen1(xraw[p][b]);
                        const float dv = (MODE == MODE_GATHER && a.m) ? __fsub_rn(xv, mk[p]) : xv;
                        const bool kept = MODE == MODE_DENSE ? (b < B) : (((km[p] >> b) & 1u) != 0);
                        unsigned short part[3];
                        split_parts<BF16>(kept ? dv : 0.0f, part);
#pragma unroll
                        for (int q = 0; q < NSPLIT; ++q) s_xh[((q * BT + b) * XLD2) * 2 + pos] = part[q];
                    }
                }
            }
        }
        __syncthreads();
        // The last block of 16 is completed with copies of the last kept row and zero activations, so that the
        // streaming loop needs no per-row predicate (a padded row adds exactly 0 for finite weights).
        const int cnt_pad = (cnt + 15) & ~15;
        if (tid < 16 && cnt > 0 && cnt + tid < cnt_pad) {
            s_k[cnt + tid] = s_k[cnt - 1];
#pragma unroll
            for (int q = 0; q < NSPLIT; ++q)
#pragma unroll
                for (int b = 0; b < BT; ++b)
                    if (b < Bp) s_xh[((q * BT + b) * XLD2) * 2 + cnt + tid] = 0;
        }
        __syncthreads();

        // ---- stream blocks of 16 kept rows; two register groups of G blocks alternate (one consumed, one in flight)
        {
            const int nblk = cnt_pad >> 4;
            const int nq = nblk > rw ? (nblk - rw + NRW - 1) / NRW : 0;  // blocks rw, rw+NRW, ...
            uint4 ga[G][4], gb[G][4];
#pragma unroll
            for (int u = 0; u < G; ++u)
#pragma unroll
                for (int r = 0; r < 4; ++r) ga[u][r] = gb[u][r] = make_uint4(0, 0, 0, 0);
            auto load_block = [&](uint4(&dst)[4], int q) {
                if (q < nq && col_ok) {  // q < nq is warp-uniform; lanes outside the matrix keep their zeros
                    const int i0 = 16 * (rw + NRW * q) + 2 * t;
                    dst[0] = ld_stream16(Wb + (size_t)s_k[i0] * row_bytes);
                    dst[1] = ld_stream16(Wb + (size_t)s_k[i0 + 1] * row_bytes);
                    dst[2] = ld_stream16(Wb + (size_t)s_k[i0 + 8] * row_bytes);
                    dst[3] = ld_stream16(Wb + (size_t)s_k[i0 + 9] * row_bytes);
                }
            };
            auto use_block = [&](const uint4(&src)[4], int q) {
                if (q >= nq) return;  // warp-uniform
                // B fragments: pair rows (2t, 2t+1) and (2t+8, 2t+9) column by column
                uint32_t b0[8], b1[8];
                const uint32_t r0[4] = {src[0].x, src[0].y, src[0].z, src[0].w}, r1[4] = {src[1].x, src[1].y, src[1].z, src[1].w};
                const uint32_t r2[4] = {src[2].x, src[2].y, src[2].z, src[2].w}, r3[4] = {src[3].x, src[3].y, src[3].z, src[3].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    b0[2 * i] = __byte_perm(r0[i], r1[i], 0x5410);
                    b0[2 * i + 1] = __byte_perm(r0[i], r1[i], 0x7632);
                    b1[2 * i] = __byte_perm(r2[i], r3[i], 0x5410);
                    b1[2 * i + 1] = __byte_perm(r2[i], r3[i], 0x7632);
                }
                const int w0 = 8 * (rw + NRW * q) + t;  // pair index of kept rows (2t, 2t+1) of this block
                if constexpr (ROWS == 8) {
                    // The 16 rows of M hold two parts of the 8 batch rows: the last part (bf16: lo) goes alone, with a
                    // zero upper half; then hi in rows 0-7 and the second part in rows 8-15 of one MMA.  Accumulator
                    // rows g hold hi (+ lo), rows g + 8 the second part; they are added when the fragments are stored.
                    if constexpr (NSPLIT == 3) {
                        const uint32_t *pl = s_xp + 2 * BT * XLD2;
                        uint32_t af[4] = {0u, 0u, 0u, 0u};
                        if (g < Bp) {
                            af[0] = pl[g * XLD2 + w0];
                            af[2] = pl[g * XLD2 + w0 + 4];
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) mma_k16<BF16>(acc[i], af, b0[i], b1[i]);
                    }
                    uint32_t af[4] = {0u, 0u, 0u, 0u};
                    if (g < Bp) {
                        af[0] = s_xp[g * XLD2 + w0];
                        af[2] = s_xp[g * XLD2 + w0 + 4];
                        af[1] = s_xp[(BT + g) * XLD2 + w0];
                        af[3] = s_xp[(BT + g) * XLD2 + w0 + 4];
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) mma_k16<BF16>(acc[i], af, b0[i], b1[i]);
                } else {
#pragma unroll
                    for (int qs = NSPLIT - 1; qs >= 0; --qs) {  // smallest part first
                        const uint32_t *pl = s_xp + qs * BT * XLD2;
                        uint32_t af[4] = {0u, 0u, 0u, 0u};
                        if (g < Bp) {
                            af[0] = pl[g * XLD2 + w0];
                            af[2] = pl[g * XLD2 + w0 + 4];
                        }
                        if (g + 8 < Bp) {
                            af[1] = pl[(g + 8) * XLD2 + w0];
                            af[3] = pl[(g + 8) * XLD2 + w0 + 4];
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i) mma_k16<BF16>(acc[i], af, b0[i], b1[i]);
                    }
                }
            };
#pragma unroll
            for (int u = 0; u < G; ++u) load_block(ga[u], u);
#pragma unroll
            for (int u = 0; u < G; ++u) load_block(gb[u], G + u);
            for (int q0 = 0; q0 < nq; q0 += 2 * G) {
#pragma unroll
                for (int u = 0; u < G; ++u) use_block(ga[u], q0 + u);
#pragma unroll
                for (int u = 0; u < G; ++u) load_block(ga[u], q0 + 2 * G + u);
#pragma unroll
                for (int u = 0; u < G; ++u) use_block(gb[u], q0 + G + u);
#pragma unroll
                for (int u = 0; u < G; ++u) load_block(gb[u], q0 + 3 * G + u);
            }
        }
        __syncthreads();
    }

    // ---- accumulator fragments -> s_red[rw][b][column]; MMA i holds columns {8 g' + i} of the chunk, and in its
    // D fragment this lane has batch rows g and g + 8 at fragment columns 2t and 2t + 1 (g' = 2t, 2t + 1).
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c0 = cw * 64 + 8 * (2 * t) + i, c1 = c0 + 8;
        if constexpr (ROWS == 16) {
            s_red[(rw * BT + g) * TNT + c0] = acc[i][0];
            s_red[(rw * BT + g) * TNT + c1] = acc[i][1];
            s_red[(rw * BT + g + 8) * TNT + c0] = acc[i][2];
            s_red[(rw * BT + g + 8) * TNT + c1] = acc[i][3];
        } else {  // rows g + 8 of the accumulator hold the second part of batch row g
            s_red[(rw * BT + g) * TNT + c0] = acc[i][0] + acc[i][2];
            s_red[(rw * BT + g) * TNT + c1] = acc[i][1] + acc[i][3];
        }
    }
    __syncthreads();
    // this CTA's partial tile, row groups added in order; s_gather is used as [b][column] here
    for (int i = tid; i < BT * TNT; i += FC_THREADS) {
        float v = 0.0f;
#pragma unroll
        for (int q = 0; q < NRW; ++q) v += s_red[q * BT * TNT + i];
        s_gather[i] = v;
    }
    // ---- cluster exchange, pull form: with up to 16 batch rows a rank owns per * B results, each the sum of S
    // partials; it reads them from its peers' shared memory (S independent loads in flight per result) in rank
    // order.  The second barrier keeps every partial tile alive until all peers have read it.
    cg::cluster_group cluster = cg::this_cluster();
    if (S > 1) cluster.sync();
    else __syncthreads();
    const float *peer[MAX_CLUSTER];
#pragma unroll
    for (int q = 0; q < MAX_CLUSTER; ++q) peer[q] = (S > 1 && q < S) ? cluster.map_shared_rank(s_gather, q) : s_gather;
    for (int it = 0; tid + it * FC_THREADS < per * B; ++it) {
        const int i = tid + it * FC_THREADS;
        const int b = i / per, c = i - b * per;
        const int row = a.out_rows ? __ldcg(a.out_rows + b) : b;
        if constexpr (EPI == EPI_BIAS) {
            const int n = tile * TNT + s * per + c;
            if (s * per + c < TNT && n < a.Nh) {
                float part[MAX_CLUSTER];
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q) part[q] = q < S ? peer[q][b * TNT + s * per + c] : 0.0f;
                float v = it == 0 ? bias0[0] : it == 1 ? bias0[1] : load_bias<BF16>(a, n);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) v += part[q];
                store_result(a, row, b, n, v);
            }
        } else {
            const int F = a.Nh, f = tile * HALF + s * per + c;
            if (s * per + c < HALF && f < F) {
                float pg[MAX_CLUSTER], pu[MAX_CLUSTER];
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q) {
                    pg[q] = q < S ? peer[q][b * TNT + s * per + c] : 0.0f;
                    pu[q] = q < S ? peer[q][b * TNT + HALF + s * per + c] : 0.0f;
                }
                float gt = it == 0 ? bias0[0] : it == 1 ? bias0[1] : (a.bias ? __ldcg(a.bias + f) : 0.0f);
                float up = it == 0 ? bias1[0] : it == 1 ? bias1[1] : (a.bias ? __ldcg(a.bias + F + f) : 0.0f);
#pragma unroll
                for (int q = 0; q < MAX_CLUSTER; ++q)
                    if (q < S) {
                        gt += pg[q];
                        up += pu[q];
                    }
                const float z = up * (gt / (1.0f + expf(-gt)));  // up * silu(gate)
                a.y[(size_t)row * a.y_ld + f] = z;
                if (a.z_copy) a.z_copy[(size_t)b * F + f] = z;
            }
        }
    }
    if (S > 1) cluster.sync();
}

template <bool BF16, int BT, int MODE, typename XT, int EPI, int TNT, int PUT = fc_pu(BT), int WB = 2>
__global__ void __launch_bounds__(FC_THREADS, fc_min_blocks(BT)) fc_kernel(const FcArgs a) {
    if constexpr (is_mma(BT)) {
        if (a.hold_dependents) {  // as below
            griddep_wait();
            fc_body_mma<BF16, BT, MODE, XT, EPI, TNT>(a, blockIdx.x, blockIdx.y, false);
        } else {
            fc_body_mma<BF16, BT, MODE, XT, EPI, TNT>(a, blockIdx.x, blockIdx.y, true);
        }
    } else if (a.hold_dependents) {  // parameter-producing call: ordinary stream order on both sides
        griddep_wait();
        fc_body<BF16, BT, MODE, XT, EPI, TNT, PUT, WB>(a, blockIdx.x, blockIdx.y, false);
    } else {
        fc_body<BF16, BT, MODE, XT, EPI, TNT, PUT, WB>(a, blockIdx.x, blockIdx.y, true);
    }
}

// ---- host-side plumbing shared by the entry points ------------------------------------------------

inline int batch_tile(int B) { return B <= 1 ? 1 : B <= 2 ? 2 : B <= 8 ? 8 : 16; }  // 3..16 rows: tensor-core variants
// Batch tile of the plain FC and FFN calls: batches up to the tuned limit stay on the fp32-FMA body.
inline int fc_batch_tile(int B) { return (B > 2 && B <= g_tune.fma_rows) ? 4 : batch_tile(B); }
inline int fc_tiles(int Nh, int epi, int tn) { return epi == EPI_GLU ? (Nh + tn / 2 - 1) / (tn / 2) : (Nh + tn - 1) / tn; }

// Tile width (256 or 128 columns) and split-K factor (cluster size) for an FC with Nh columns per half and
// `groups` concurrently active groups (experts): the pair with the most CTAs that are still all co-resident.
void choose_config(int K, int Nh, int epi, int groups, int B, int *tn, int *S);
int resident_ctas(int S);  // CTAs of clusters of size S resident at once (256 threads, two CTAs per SM)

// tcgen05 kernel for batch 3..16 (scap_fc_tc.cu): whether it can take this call, its split-K factor, its launch,
// and the status word of its bounded waits (0 = none ran out; reading synchronises the device and clears it).
bool tc_applicable(const FcArgs &a, int epi, bool bf16);
int tc_choose_split(int K, int Nh, int epi, int B, bool bf16);
cudaError_t launch_fc_tc(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st);
int tc_take_status();
// Dense-stream tcgen05 kernel (scap_fc_tc.cu): TMA box loads of all rows, pruning on the activation operand.
bool ds_applicable(const FcArgs &a, int epi, bool bf16);
int ds_choose_split(int K, int Nh, int epi);
cudaError_t launch_fc_ds(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st);
int *tc_status_ptr();  // device address of that status word on the current device (NULL if it cannot be had)

// Launch with cluster dimension (1, S, 1) and, if enabled, programmatic dependent launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, int cluster_y,
                                  cudaStream_t stream, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = cluster_y;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster_y > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// xkind: 0 fp16, 1 bf16, 2 fp32 activations.
cudaError_t launch_fc(bool bf16, int mode, int xkind, int epi, const FcArgs &a, cudaStream_t st);

// Inspection helper: expands the union keep mask into the ascending list of kept channels (one CTA).
cudaError_t launch_expand_bits(const uint32_t *bits, int K, uint32_t *idx_out, int *nnz_out, cudaStream_t st);

}  // namespace scap
