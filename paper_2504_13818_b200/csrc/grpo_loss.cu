// grpo_loss: the GRPO-PODS token objective L_PODS(theta, S) of Section 3.2 and its gradient with
// respect to the bf16 logits, fused: per row the softmax statistics and the target log-prob, the
// scalar loss terms, then the gradient row.
//
// grpo_loss_chunk picks one of three kernels by the row shape: the cluster-resident pipeline
// (grpo_loss_cluster.cu) for long aligned rows, the row-tile kernel below for short aligned rows, and
// the general row kernel for everything else (any V, any pitch or alignment).
//
// Row kernel (one CTA per row at a time, persistent over rows), three uniform sweeps of the row:
//   max   128-bit loads from HBM, packed bf16x2 maxima; each thread remembers where its maximum
//         was; a block arg-max gives the row maximum M and the position of its first instance;
//   sum   the row again (just read: served by L2): sum of 2^(x log2e - ref), ref = fl(M log2e),
//         over every element EXCEPT that one instance of the maximum, so that a row dominated by
//         one logit keeps full relative accuracy in Z - 1 (hence in 1 - p of the dominating token);
//         the exact residual M log2e - ref is applied to the finished sum as the factor 2^(-lo);
//   scalar  one thread, fp64: logp, rho, clipped surrogate, KL term, the row factor g_t, and the
//         row's weighted loss term into the workspace;
//   grad  the row a third time (L2): write bf16(g_t (onehot - softmax)).  Rows whose g_t is exactly
//         0 (masked, or clipped with no KL term) are written as zeros without being re-read.
// No sweep has a data-dependent branch except at the one vector holding the excluded maximum.
// Loss reduction: a single CTA sums the chunk's per-row terms in a fixed order (deterministic).

#include "grpo_loss_common.cuh"

using namespace pods_loss;

namespace {

constexpr int kBatch = 4;          // 128-bit loads in flight per thread

struct RowShared {
    unsigned long long red_k[32];
    double red_d[32];
    float row_max;
    int max_pos;        // position code of the first instance of the maximum
    double zprime;      // sum over the row of 2^(x log2e - ref), one instance of the maximum excluded
    float coef;         // -g_t / Z (with the reference correction)
    float target;       // g_t (1 - p_token)
    int write_mode;     // 0: zeros, 1: gradient
    int token;
};

__device__ __forceinline__ uint4 ld_global_v4(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// One batch of kBatch vectors, BLOCK apart, starting at vector v0 (missing ones read as -inf).
template <int BLOCK>
__device__ __forceinline__ void load_batch(uint4 (&q)[kBatch], const uint4* row4, int v0, int nvec) {
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
        const int v = v0 + j * BLOCK;
        q[j] = v < nvec ? ld_global_v4(row4 + v) : make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);
    }
}

__device__ __forceinline__ float vec_sum_ex2(const uint4& q, float ref) {
    const float a = ex2_approx(fmaf(bf16_lo(q.x), kLog2e, -ref)) + ex2_approx(fmaf(bf16_hi(q.x), kLog2e, -ref));
    const float b = ex2_approx(fmaf(bf16_lo(q.y), kLog2e, -ref)) + ex2_approx(fmaf(bf16_hi(q.y), kLog2e, -ref));
    const float c = ex2_approx(fmaf(bf16_lo(q.z), kLog2e, -ref)) + ex2_approx(fmaf(bf16_hi(q.z), kLog2e, -ref));
    const float d = ex2_approx(fmaf(bf16_lo(q.w), kLog2e, -ref)) + ex2_approx(fmaf(bf16_hi(q.w), kLog2e, -ref));
    return (a + b) + (c + d);
}

// The vector that holds the excluded instance: every element but the first one equal to mx.
__device__ __forceinline__ float ex2_unless(float x, float ref, float mx, bool& skipped) {
    const bool skip = !skipped && x == mx;
    skipped |= skip;
    return skip ? 0.0f : ex2_approx(fmaf(x, kLog2e, -ref));
}

__device__ __noinline__ float vec_sum_ex2_excluding(uint4 q, float ref, float mx) {
    bool skipped = false;
    float s = ex2_unless(bf16_lo(q.x), ref, mx, skipped);
    s += ex2_unless(bf16_hi(q.x), ref, mx, skipped);
    s += ex2_unless(bf16_lo(q.y), ref, mx, skipped);
    s += ex2_unless(bf16_hi(q.y), ref, mx, skipped);
    s += ex2_unless(bf16_lo(q.z), ref, mx, skipped);
    s += ex2_unless(bf16_hi(q.z), ref, mx, skipped);
    s += ex2_unless(bf16_lo(q.w), ref, mx, skipped);
    s += ex2_unless(bf16_hi(q.w), ref, mx, skipped);
    return s;
}

__device__ __forceinline__ uint4 grad_vec(const uint4& q, float coef, float ref) {
    uint4 o;
    o.x = pack_bf16x2(coef * ex2_approx(fmaf(bf16_lo(q.x), kLog2e, -ref)),
                      coef * ex2_approx(fmaf(bf16_hi(q.x), kLog2e, -ref)));
    o.y = pack_bf16x2(coef * ex2_approx(fmaf(bf16_lo(q.y), kLog2e, -ref)),
                      coef * ex2_approx(fmaf(bf16_hi(q.y), kLog2e, -ref)));
    o.z = pack_bf16x2(coef * ex2_approx(fmaf(bf16_lo(q.z), kLog2e, -ref)),
                      coef * ex2_approx(fmaf(bf16_hi(q.z), kLog2e, -ref)));
    o.w = pack_bf16x2(coef * ex2_approx(fmaf(bf16_lo(q.w), kLog2e, -ref)),
                      coef * ex2_approx(fmaf(bf16_hi(q.w), kLog2e, -ref)));
    return o;
}

// Block arg-max: the largest value, and among equal values the smallest position code.
template <int BLOCK>
__device__ __forceinline__ void block_argmax(float v, int pos, RowShared& sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long key = argmax_key(v, pos);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(PODS_FULL_MASK, key, d);
        key = o > key ? o : key;
    }
    if (lane == 0) sh.red_k[warp] = key;
    __syncthreads();
    if (warp == 0) {
        unsigned long long k = lane < BLOCK / 32 ? sh.red_k[lane] : 0ull;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const unsigned long long o = __shfl_xor_sync(PODS_FULL_MASK, k, d);
            k = o > k ? o : k;
        }
        if (lane == 0) {
            sh.row_max = argmax_key_value(k);
            sh.max_pos = argmax_key_pos(k);
        }
    }
    __syncthreads();
}

template <int BLOCK>
__device__ __forceinline__ void block_sum(double v, RowShared& sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(PODS_FULL_MASK, v, d);
    if (lane == 0) sh.red_d[warp] = v;
    __syncthreads();
    if (warp == 0) {
        double w = lane < BLOCK / 32 ? sh.red_d[lane] : 0.0;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) w += __shfl_xor_sync(PODS_FULL_MASK, w, d);
        if (lane == 0) sh.zprime = w;
    }
    __syncthreads();
}

template <int BLOCK>
__global__ void __launch_bounds__(BLOCK, 2048 / BLOCK / 2)
grpo_loss_rows_kernel(const RowArgs a) {
    __shared__ RowShared sh;
    const int tid = threadIdx.x;
    const int V = a.V;
    const int nvec = a.vec_ok ? V / 8 : 0;
    const int tail0 = nvec * 8;
    // Position codes: vector v -> v, tail element e -> nvec + (e - tail0).

    for (int64_t t = blockIdx.x; t < a.T; t += gridDim.x) {
        const uint16_t* row = a.logits + t * a.ldl;
        uint16_t* drow = a.dlogits + t * a.ldd;
        const uint4* row4 = reinterpret_cast<const uint4*>(row);

        float x_tok = 0.0f;
        if (tid == 0) {
            int tok = a.tokens[t];
            if (tok < 0 || tok >= V) { tok = 0; pods_raise(a.status, PODS_STATUS_TOKEN_RANGE); }
            sh.token = tok;
            x_tok = __uint_as_float((uint32_t)row[tok] << 16);   // read before anything is written in place
        }

        // ---- sweep 1: maximum and where it is ----------------------------------------------
        // (every sweep keeps the next batch of loads in flight while it works on the current one)
        float m_t = -INFINITY;
        int pos_t = 0x7fffffff;
        {
            uint4 nxt[kBatch];
            load_batch<BLOCK>(nxt, row4, tid, nvec);
            for (int v0 = tid; v0 < nvec; v0 += kBatch * BLOCK) {
                uint4 q[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) q[j] = nxt[j];
                if (v0 + kBatch * BLOCK < nvec) load_batch<BLOCK>(nxt, row4, v0 + kBatch * BLOCK, nvec);
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const float vm = vec_max(q[j]);
                    if (vm > m_t) { m_t = vm; pos_t = v0 + j * BLOCK; }
                }
            }
        }
        for (int e = tail0 + tid; e < V; e += BLOCK) {
            const float x = __uint_as_float((uint32_t)row[e] << 16);
            if (x > m_t) { m_t = x; pos_t = nvec + (e - tail0); }
        }
        block_argmax<BLOCK>(m_t, pos_t, sh);
        const float mx = sh.row_max;
        const int excl = sh.max_pos;
        const float ref = mx * kLog2e;

        // ---- sweep 2: sum of exponentials, one instance of the maximum left out ---------------
        float s_t = 0.0f;
        if (a.precise) {
            // small chunk: e^(x - M) in fp64, no reference exponent and no correction factor
            double sd = 0.0;
            for (int v = tid; v < nvec; v += BLOCK) sd += exact_exp_sum(ld_global_v4(row4 + v), mx, v == excl);
            for (int e = tail0 + tid; e < V; e += BLOCK) {
                const float x = __uint_as_float((uint32_t)row[e] << 16);
                if (nvec + (e - tail0) != excl && x != -INFINITY) sd += exp((double)x - (double)mx);
            }
            block_sum<BLOCK>(sd, sh);
        } else {
        {
            uint4 nxt[kBatch];
            load_batch<BLOCK>(nxt, row4, tid, nvec);
            for (int v0 = tid; v0 < nvec; v0 += kBatch * BLOCK) {
                uint4 q[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) q[j] = nxt[j];
                if (v0 + kBatch * BLOCK < nvec) load_batch<BLOCK>(nxt, row4, v0 + kBatch * BLOCK, nvec);
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    if (v0 + j * BLOCK == excl) s_t += vec_sum_ex2_excluding(q[j], ref, mx);
                    else s_t += vec_sum_ex2(q[j], ref);              // padding is -inf: adds 0
                }
            }
        }
        for (int e = tail0 + tid; e < V; e += BLOCK) {
            const float x = __uint_as_float((uint32_t)row[e] << 16);
            if (nvec + (e - tail0) != excl) s_t += ex2_approx(fmaf(x, kLog2e, -ref));
        }
        block_sum<BLOCK>((double)s_t, sh);
        }

        // ---- scalar terms of the row (one thread, fp64) ---------------------------------------
        if (tid == 0) {
            const double corr = ref_correction(mx, ref);
            const RowInputs in = load_row_inputs(a, t);
            const RowScalars r = row_scalars(a, in, x_tok, mx, a.precise ? sh.zprime : sh.zprime * corr);
            a.logp[t] = (float)r.logp;
            a.row_loss[t] = r.weighted_loss;
            sh.coef = (float)(-r.g / r.Z * corr);
            sh.target = (float)(r.g * r.one_minus_p);
            sh.write_mode = (r.g != 0.0) ? 1 : 0;
        }
        __syncthreads();

        // ---- sweep 3: the gradient row --------------------------------------------------------
        const int tok = sh.token;
        uint4* d4 = reinterpret_cast<uint4*>(drow);
        if (sh.write_mode == 0) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            for (int v = tid; v < nvec; v += BLOCK) __stcs(d4 + v, z);
            for (int e = tail0 + tid; e < V; e += BLOCK) drow[e] = 0;
        } else {
            const float coef = sh.coef;
            const uint16_t target_bits = to_bf16_bits(sh.target);
            const int tok_vec = tok >> 3;
            uint4 nxt[kBatch];
            load_batch<BLOCK>(nxt, row4, tid, nvec);
            for (int v0 = tid; v0 < nvec; v0 += kBatch * BLOCK) {
                uint4 q[kBatch];
#pragma unroll
                for (int j = 0; j < kBatch; ++j) q[j] = nxt[j];
                if (v0 + kBatch * BLOCK < nvec) load_batch<BLOCK>(nxt, row4, v0 + kBatch * BLOCK, nvec);
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int v = v0 + j * BLOCK;
                    if (v < nvec && PODS_INDEX_OK((int64_t)v * 8 + 7, a.ldd, a.status)) {
                        uint4 o = grad_vec(q[j], coef, ref);
                        if (v == tok_vec) patch_bf16(o, tok & 7, target_bits);
                        __stcs(d4 + v, o);
                    }
                }
            }
            for (int e = tail0 + tid; e < V; e += BLOCK) {
                const float x = __uint_as_float((uint32_t)row[e] << 16);
                drow[e] = (e == tok) ? target_bits : to_bf16_bits(coef * ex2_approx(fmaf(x, kLog2e, -ref)));
            }
        }
        __syncthreads();     // sh is reused by the next row
    }
}

// Fixed-order sum of the chunk's per-row loss terms, added to the accumulator.
__global__ void __launch_bounds__(1024)
loss_reduce_kernel(const double* __restrict__ row_loss, int64_t T, double* loss_acc) {
    __shared__ double part[1024];
    double s = 0.0;
    for (int64_t t = threadIdx.x; t < T; t += 1024) s += row_loss[t];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int d = 512; d > 0; d >>= 1) {
        if ((int)threadIdx.x < d) part[threadIdx.x] += part[threadIdx.x + d];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss_acc += part[0];
}

__global__ void loss_zero_kernel(double* loss_acc) { *loss_acc = 0.0; }

__global__ void loss_finalize_kernel(const double* loss_acc, float* loss) { *loss = (float)*loss_acc; }


// ---------------------------------------------------------------------------------------------
// Row-tile kernel for short rows (V <= 4096, V % 8 == 0, 16-byte aligned rows).
// ---------------------------------------------------------------------------------------------
// A row of a small vocabulary is only a few KB: one CTA per row leaves most of its threads idle and
// pays the fp64 scalar terms once per row on a single thread.  Here a CTA of eight warps takes a tile
// of R rows (R * V * 2 bytes <= 64 KB of shared memory); one WARP owns a whole row:
//   A  row -> registers with 128-bit loads, packed maxima, warp arg-max, e = 2^(x log2e - ref) summed
//      with one instance of the maximum left out, bf16(e) parked in the tile;
//   B  the first R threads of the CTA evaluate the fp64 scalar terms of one row each, side by side;
//   C  each warp turns its rows' e into bf16(coef e) and stores them, then fixes the target entry.
// HBM sees one read and one write per element; the exponential is taken once.
constexpr int kTileWarps = 8;
constexpr int kTileMaxRows = 64;
constexpr int kTileBytes = 64 * 1024;

template <int IT, bool EXACT_SUM>
__global__ void __launch_bounds__(kTileWarps * 32)
grpo_loss_tile_kernel(const RowArgs a, const int rows_per_tile) {
    extern __shared__ __align__(16) uint4 tile[];
    __shared__ float s_mx[kTileMaxRows], s_sum[kTileMaxRows], s_coef[kTileMaxRows], s_target[kTileMaxRows];
    __shared__ double s_sum_exact[EXACT_SUM ? kTileMaxRows : 1];
    __shared__ int s_mode[kTileMaxRows], s_tok[kTileMaxRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec = a.V / 8;
    const uint4 neg_inf4 = make_uint4(kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair);

    for (int64_t tile0 = (int64_t)blockIdx.x * rows_per_tile; tile0 < a.T; tile0 += (int64_t)gridDim.x * rows_per_tile) {
        const int n_rows = (int)(a.T - tile0 < rows_per_tile ? a.T - tile0 : rows_per_tile);

        // ---- A: statistics of my rows; e parked in the tile --------------------------------------------
        for (int r = warp; r < n_rows; r += kTileWarps) {
            const uint4* row4 = reinterpret_cast<const uint4*>(a.logits + (tile0 + r) * a.ldl);
            uint4 q[IT];
#pragma unroll
            for (int k = 0; k < IT; ++k) {
                const int j = lane + 32 * k;
                q[k] = j < nvec ? row4[j] : neg_inf4;
            }
            uint32_t pm[4] = {kNegInfPair, kNegInfPair, kNegInfPair, kNegInfPair};
#pragma unroll
            for (int k = 0; k < IT; ++k) max_vec(pm, q[k]);
            const uint32_t pmax = max_bf16x2(max_bf16x2(pm[0], pm[1]), max_bf16x2(pm[2], pm[3]));
            const float m_t = fmaxf(bf16_lo(pmax), bf16_hi(pmax)) + 0.0f;             // -0 -> +0
            const uint32_t key_w = __reduce_max_sync(PODS_FULL_MASK, (ordered16(m_t) << 16) | (uint32_t)(31 - lane));
            const float mx = from_ordered16(key_w >> 16);
            const int owner = 31 - (int)(key_w & 0xffffu);               // lowest lane that holds an instance of the maximum
            const float ref = mx == -INFINITY ? 0.0f : mx * kLog2e;
            int excl = -1;                                               // the owner's first vector that holds it
            if (lane == owner) {
#pragma unroll
                for (int k = IT - 1; k >= 0; --k)
                    if (vec_max(q[k]) == mx) excl = k;
            }
            if (EXACT_SUM) {
                double sd = 0.0;
#pragma unroll
                for (int k = 0; k < IT; ++k) sd += exact_exp_sum(q[k], mx, k == excl);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) sd += __shfl_xor_sync(PODS_FULL_MASK, sd, d);
                if (lane == 0) s_sum_exact[r] = sd;
            }
            float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
            for (int k = 0; k < IT; ++k) {
                const int j = lane + 32 * k;
                const float part = (k == excl) ? exp_sum_excluding(q[k], ref, mx) : 0.0f;
                const float sum = exp_vec_inplace(q[k], ref);
                if (k & 1) s1 += (k == excl) ? part : sum; else s0 += (k == excl) ? part : sum;
                if (j < nvec && PODS_INDEX_OK((size_t)r * nvec + j, (size_t)rows_per_tile * nvec, a.status)) tile[(size_t)r * nvec + j] = q[k];
            }
            float sw = s0 + s1;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) sw += __shfl_xor_sync(PODS_FULL_MASK, sw, d);
            if (lane == 0) { s_mx[r] = mx; s_sum[r] = sw; }
        }
        __syncthreads();

        // ---- B: the scalar terms, one row per thread ---------------------------------------------------------
        if (tid < n_rows) {
            const int64_t t = tile0 + tid;
            int tok = a.tokens[t];
            if (tok < 0 || tok >= a.V) { tok = 0; pods_raise(a.status, PODS_STATUS_TOKEN_RANGE); }
            const float x_tok = __uint_as_float((uint32_t)a.logits[t * a.ldl + tok] << 16);   // before phase C stores this row in place
            const float mx = s_mx[tid];
            const double corr = ref_correction(mx, mx * kLog2e);
            const RowInputs in = load_row_inputs(a, t);
            // the gradient rows scale the stored e = 2^(x log2e - ref): their factor keeps the correction either way
            const RowScalars r = row_scalars(a, in, x_tok, mx, EXACT_SUM ? s_sum_exact[tid] : (double)s_sum[tid] * corr);
            a.logp[t] = (float)r.logp;
            a.row_loss[t] = r.weighted_loss;
            s_coef[tid] = (float)(-r.g / r.Z * corr);
            s_target[tid] = (float)(r.g * r.one_minus_p);
            s_mode[tid] = (r.g != 0.0) ? 1 : 0;
            s_tok[tid] = tok;
        }
        __syncthreads();

        // ---- C: the gradient rows ---------------------------------------------------------------------------
        for (int r = warp; r < n_rows; r += kTileWarps) {
            uint4* out = reinterpret_cast<uint4*>(a.dlogits + (tile0 + r) * a.ldd);
            if (s_mode[r] == 0) {
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                for (int j = lane; j < nvec; j += 32) out[j] = z;
                continue;
            }
            const float coef = s_coef[r];
            const uint16_t hi16 = to_bf16_bits(coef);
            const uint16_t lo16 = to_bf16_bits(coef - __uint_as_float((uint32_t)hi16 << 16));
            const uint32_t c_hi = (uint32_t)hi16 * 0x10001u, c_lo = (uint32_t)lo16 * 0x10001u;
#pragma unroll
            for (int k = 0; k < IT; ++k) {
                const int j = lane + 32 * k;
                if (j < nvec && PODS_INDEX_OK((size_t)r * nvec + j, (size_t)rows_per_tile * nvec, a.status) &&
                    PODS_INDEX_OK(tile0 + r, a.T, a.status)) {
                    uint4 e = tile[(size_t)r * nvec + j];
                    scale_vec(e, c_hi, c_lo);
                    out[j] = e;
                }
            }
            const int tok = s_tok[r];
            if (((tok >> 3) & 31) == lane)                               // rewritten by the lane that stored its vector
                reinterpret_cast<uint16_t*>(out)[tok] = to_bf16_bits(s_target[r]);
        }
        __syncthreads();                                                 // the tile and the row slots are reused
    }
}

template <int IT, bool EXACT_SUM>
int launch_tile_as(const RowArgs& a, cudaStream_t s) {
    const int nvec = a.V / 8;
    int rows = kTileBytes / (nvec * 16);
    rows = rows > kTileMaxRows ? kTileMaxRows : rows & ~(kTileWarps - 1);
    // a small chunk is spread over the whole GPU: fewer rows per tile, more tiles
    if (EXACT_SUM) {
        const int64_t spread = (a.T + pods_sm_count() - 1) / pods_sm_count();
        const int want = (int)((spread + kTileWarps - 1) / kTileWarps * kTileWarps);
        rows = want < rows ? want : rows;
    }
    const size_t smem = (size_t)rows * nvec * 16;
    auto kernel = grpo_loss_tile_kernel<IT, EXACT_SUM>;
    PODS_RETURN_IF_CUDA_ERROR(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t tiles = (a.T + rows - 1) / rows;
    const int64_t cap = (int64_t)pods_sm_count() * 3;
    kernel<<<(unsigned)(tiles < cap ? tiles : cap), kTileWarps * 32, smem, s>>>(a, rows);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

template <int IT>
int launch_tile(const RowArgs& a, cudaStream_t s) {
    return a.precise ? launch_tile_as<IT, true>(a, s) : launch_tile_as<IT, false>(a, s);
}

// Short rows on the row-tile kernel; *launched says whether the shape was taken.
int launch_grpo_loss_tile(const RowArgs& a, cudaStream_t s, bool* launched) {
    *launched = false;
    if (!a.vec_ok || a.V % 8 != 0 || a.V > 4096) return PODS_OK;
    *launched = true;
    const int it = (a.V / 8 + 31) / 32;
    if (it <= 1) return launch_tile<1>(a, s);
    if (it <= 2) return launch_tile<2>(a, s);
    if (it <= 4) return launch_tile<4>(a, s);
    if (it <= 8) return launch_tile<8>(a, s);
    return launch_tile<16>(a, s);
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

int pods_loss::launch_loss_reduce(const double* row_loss, int64_t T, double* loss_acc, cudaStream_t stream) {
    loss_reduce_kernel<<<1, 1024, 0, stream>>>(row_loss, T, loss_acc);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

extern "C" size_t grpo_loss_chunk_workspace_bytes(int64_t T_chunk) {
    if (T_chunk < 0) return 0;
    return align_up((size_t)T_chunk * sizeof(double), 256) + align_up((size_t)T_chunk * sizeof(RowPrep), 256) + 256;
}

extern "C" int grpo_loss_chunk(const void* logits, int64_t ldl, const int32_t* tokens, const float* old_logp,
                               const float* ref_logp, const float* adv, const double* seq_weight,
                               const int64_t* cu_seqlens, int64_t M, int64_t row0, const uint8_t* mask,
                               int64_t T_chunk, int32_t V, float eps, float beta, float grad_scale,
                               double* loss_acc, float* logp, void* dlogits, int64_t ldd, void* workspace,
                               size_t workspace_bytes, uint32_t* status, void* stream) {
    if (T_chunk < 0 || V < 1 || M < 1 || row0 < 0 || ldl < V || ldd < V) return PODS_ERR_INVALID_ARG;
    if (!(eps >= 0.0f) || !(beta == beta)) return PODS_ERR_INVALID_ARG;
    if (T_chunk == 0) return PODS_OK;
    if (logits == nullptr || tokens == nullptr || old_logp == nullptr || adv == nullptr || seq_weight == nullptr ||
        cu_seqlens == nullptr || loss_acc == nullptr || logp == nullptr || dlogits == nullptr)
        return PODS_ERR_INVALID_ARG;
    if (ref_logp == nullptr && beta != 0.0f) return PODS_ERR_INVALID_ARG;
    if (!pods_aligned(logits, 2) || !pods_aligned(dlogits, 2) || !pods_aligned(loss_acc, 8)) return PODS_ERR_INVALID_ARG;
    if (dlogits == logits && ldd != ldl) return PODS_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < grpo_loss_chunk_workspace_bytes(T_chunk) ||
        !pods_aligned(workspace, 16))
        return PODS_ERR_WORKSPACE;

    RowArgs a;
    a.logits = static_cast<const uint16_t*>(logits);
    a.ldl = ldl;
    a.tokens = tokens;
    a.old_logp = old_logp;
    a.ref_logp = ref_logp;
    a.adv = adv;
    a.seq_weight = seq_weight;
    a.cu_seqlens = cu_seqlens;
    a.M = M;
    a.row0 = row0;
    a.mask = mask;
    a.T = T_chunk;
    a.V = V;
    a.eps = eps;
    a.beta = beta;
    a.grad_scale = grad_scale;
    a.logp = logp;
    a.dlogits = static_cast<uint16_t*>(dlogits);
    a.ldd = ldd;
    a.row_loss = static_cast<double*>(workspace);
    a.prep = reinterpret_cast<RowPrep*>(static_cast<unsigned char*>(workspace) + align_up((size_t)T_chunk * sizeof(double), 256));
    a.status = status;
    a.vec_ok = pods_aligned(logits, 16) && pods_aligned(dlogits, 16) && ldl % 8 == 0 && ldd % 8 == 0;
    a.precise = T_chunk * (int64_t)V <= kExactSumMaxLogits;

    cudaStream_t s = pods_stream(stream);
    bool on_cluster_path = false;
    const int rc_cluster = launch_grpo_loss_cluster(a, s, &on_cluster_path);
    if (rc_cluster != PODS_OK) return rc_cluster;
    if (on_cluster_path) {
        loss_reduce_kernel<<<1, 1024, 0, s>>>(a.row_loss, T_chunk, loss_acc);
        PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
        return PODS_OK;
    }
    bool on_tile_path = false;
    const int rc_tile = launch_grpo_loss_tile(a, s, &on_tile_path);
    if (rc_tile != PODS_OK) return rc_tile;
    if (on_tile_path) {
        loss_reduce_kernel<<<1, 1024, 0, s>>>(a.row_loss, T_chunk, loss_acc);
        PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
        return PODS_OK;
    }
    // one CTA per row: fewer threads for shorter rows, so that every thread has several vectors and an SM
    // holds more rows at once (1024 resident threads per SM in every case); limits from timings at
    // V = 4K .. 152K: 128 threads win up to 24576 (4.2-4.5 TB/s), 256 up to 49152 (4.3-4.4), 512 beyond (4.1)
    const int64_t sms = pods_sm_count();
    if (V <= 24576) {
        const int64_t cap = sms * 8;
        grpo_loss_rows_kernel<128><<<(int)(T_chunk < cap ? T_chunk : cap), 128, 0, s>>>(a);
    } else if (V <= 53248) {
        const int64_t cap = sms * 4;
        grpo_loss_rows_kernel<256><<<(int)(T_chunk < cap ? T_chunk : cap), 256, 0, s>>>(a);
    } else {
        const int64_t cap = sms * 2;
        grpo_loss_rows_kernel<512><<<(int)(T_chunk < cap ? T_chunk : cap), 512, 0, s>>>(a);
    }
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    loss_reduce_kernel<<<1, 1024, 0, s>>>(a.row_loss, T_chunk, loss_acc);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

extern "C" size_t grpo_loss_workspace_bytes(int64_t T, int64_t M, int64_t chunk_rows) {
    if (T < 0 || M < 0) return 0;
    const int64_t rows = (chunk_rows <= 0 || chunk_rows > T) ? T : chunk_rows;
    return grpo_loss_chunk_workspace_bytes(rows) + align_up((size_t)M * sizeof(double), 256) + 256;
}

extern "C" int grpo_loss_fwd_bwd(const void* logits, int64_t ldl, const int32_t* tokens, const float* old_logp,
                                 const float* ref_logp, const float* adv, const int64_t* cu_seqlens, int64_t M,
                                 const uint8_t* mask, int64_t T, int32_t V, float eps, float beta,
                                 int64_t chunk_rows, float* loss, float* logp, void* dlogits, int64_t ldd,
                                 void* workspace, size_t workspace_bytes, uint32_t* status, void* stream) {
    if (T < 0 || M < 1 || loss == nullptr) return PODS_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < grpo_loss_workspace_bytes(T, M, chunk_rows) ||
        !pods_aligned(workspace, 16))
        return PODS_ERR_WORKSPACE;
    const int64_t rows = (chunk_rows <= 0 || chunk_rows > T) ? T : chunk_rows;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    double* loss_acc = reinterpret_cast<double*>(ws);
    double* seq_weight = reinterpret_cast<double*>(ws + 256);
    unsigned char* chunk_ws = ws + 256 + align_up((size_t)M * sizeof(double), 256);
    const size_t chunk_ws_bytes = grpo_loss_chunk_workspace_bytes(rows);
    cudaStream_t s = pods_stream(stream);

    loss_zero_kernel<<<1, 1, 0, s>>>(loss_acc);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    int rc = grpo_seq_weights(mask, cu_seqlens, M, seq_weight, stream);
    if (rc != PODS_OK) return rc;
    const uint16_t* lg = static_cast<const uint16_t*>(logits);
    uint16_t* dl = static_cast<uint16_t*>(dlogits);
    for (int64_t r0 = 0; r0 < T; r0 += rows) {
        const int64_t cnt = (T - r0 < rows) ? T - r0 : rows;
        rc = grpo_loss_chunk(lg + r0 * ldl, ldl, tokens + r0, old_logp + r0, ref_logp ? ref_logp + r0 : nullptr,
                             adv, seq_weight, cu_seqlens, M, r0, mask ? mask + r0 : nullptr, cnt, V, eps, beta,
                             1.0f, loss_acc, logp + r0, dl + r0 * ldd, ldd, chunk_ws, chunk_ws_bytes, status,
                             stream);
        if (rc != PODS_OK) return rc;
    }
    return grpo_loss_finalize(loss_acc, loss, stream);
}

extern "C" int grpo_loss_finalize(const double* loss_acc, float* loss, void* stream) {
    if (loss_acc == nullptr || loss == nullptr) return PODS_ERR_INVALID_ARG;
    loss_finalize_kernel<<<1, 1, 0, pods_stream(stream)>>>(loss_acc, loss);
    PODS_RETURN_IF_CUDA_ERROR(cudaGetLastError());
    return PODS_OK;
}

// ---------------------------------------------------------------------------------------------
// grpo_loss_chunk_static: grpo_loss_chunk for callers that cannot hand over a workspace.
// ---------------------------------------------------------------------------------------------
// The per-row loss terms live in a fixed device array that is part of the library image, so the
// call needs no workspace argument and allocates nothing.

#define PODS_STATIC_CHUNK_ROWS 16384

namespace {

// One fp64 slot per row of the largest chunk, plus the pad the workspace size formula asks for.
constexpr size_t kStaticScratchBytes = (size_t)PODS_STATIC_CHUNK_ROWS * (sizeof(double) + sizeof(RowPrep)) + 512;
static __device__ __align__(256) unsigned char g_static_row_loss[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices] = {};     // device address of the array, per device ordinal

// The array's name is only a handle on the host; its device address has to be asked for, on the
// device that is current.  Done on the first call per device and remembered.
int static_scratch_address(void** out) {
    int dev = 0;
    PODS_RETURN_IF_CUDA_ERROR(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return PODS_ERR_UNSUPPORTED;
    void* p = __atomic_load_n(&g_static_scratch_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        PODS_RETURN_IF_CUDA_ERROR(cudaGetSymbolAddress(&p, g_static_row_loss));
        if (p == nullptr) return PODS_ERR_CUDA;
        __atomic_store_n(&g_static_scratch_ptr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return PODS_OK;
}

}  // namespace

extern "C" int64_t grpo_loss_chunk_static_max_rows(void) { return PODS_STATIC_CHUNK_ROWS; }

extern "C" int grpo_loss_chunk_static(const void* logits, int64_t ldl, const int32_t* tokens,
                                      const float* old_logp, const float* ref_logp, const float* adv,
                                      const double* seq_weight, const int64_t* cu_seqlens, int64_t M,
                                      int64_t row0, const uint8_t* mask, int64_t T_chunk, int32_t V, float eps,
                                      float beta, float grad_scale, double* loss_acc, float* logp,
                                      void* dlogits, int64_t ldd, uint32_t* status, void* stream) {
    if (T_chunk > PODS_STATIC_CHUNK_ROWS) return PODS_ERR_STATIC_CAPACITY;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != PODS_OK) return rc;
    return grpo_loss_chunk(logits, ldl, tokens, old_logp, ref_logp, adv, seq_weight, cu_seqlens, M, row0, mask,
                           T_chunk, V, eps, beta, grad_scale, loss_acc, logp, dlogits, ldd, scratch,
                           kStaticScratchBytes, status, stream);
}
