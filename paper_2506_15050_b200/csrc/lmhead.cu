// LM-head variant of the fused policy loss: logits x = hidden * weight are a dense [M,K] x [K,V]
// bf16 contraction on the tensor cores (tcgen05, fp32 accumulation in tensor memory) and are never
// written to memory.  Math per row as in Eq. 1 of the paper (see tppo_policy_loss_fwd_bwd).
//
// Passes, all built on umma_gemm_kernel with different epilogues:
//   1. statistics   x tiles -> per (row, 256-column tile) running max and sum of exponentials, plus
//                   the target logit; a row kernel merges them into the log-prob, the clipped
//                   surrogate and the gradient factor c of the row.
//   then, for each chunk of vocabulary columns (a few thousand, sized to fill whole waves of tiles):
//   2a. gradient     x tiles recomputed -> dX = c * (softmax - onehot) in bf16 into a chunk buffer
//   2b. dhidden     += dX_chunk * W_chunk^T   (fp32 accumulator in the workspace, bf16 on the last)
//   2c. dweight[:, chunk] = hidden^T * dX_chunk
// Four GEMM-sized contractions in total; the chunk buffer is the only logits-shaped memory.
#include "policy_common.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_pair.cuh"

namespace tppo {

int launch_policy_prepare(const PolicyArgs& a, cudaStream_t s);
int launch_policy_finish(const PolicyArgs& a, cudaStream_t s);

namespace {

constexpr float kInf = __builtin_huge_valf();

// ---- epilogues ------------------------------------------------------------------------------
// Pass 1: online max / sum-of-exponentials over the 256 columns of the tile, target logit.
struct EpiStats {
    const RowRec* rec;
    float2* part;      // [n_tiles][M]: (max, sum exp(x - max)) of the tile's valid columns
    float* xy;         // [M]: logit of the target token
    int64_t M;
    int32_t V;         // columns of this weight matrix (a vocabulary shard when v_off / V differ from the whole)
    int32_t v_off;     // vocabulary id of column 0
    __device__ __forceinline__ void operator()(int mt, int nt, int row, uint32_t taddr) const {
        const int64_t r = int64_t(mt) * kTileM + row;
        const int n0 = nt * kTileN;
        const int yg = r < M ? load_rec(rec + r).y : -1;
        // column of the target; far off when the row is skipped or the target lies in another shard
        const int y = (yg >= v_off && yg - v_off < V) ? yg - v_off : -1 - kTileN;
        float m = -kInf, s = 0.f, xv = 0.f;
        bool found = false;
#pragma unroll 1
        for (int c = 0; c < kTileN; c += 32) {
            const int col0 = n0 + c;
            if (col0 >= V) break;                        // uniform over the warp
            uint32_t v[32];
            umma::tmem_ld32(taddr + c, v);
            umma::tmem_ld_wait();
            float x[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) x[i] = __uint_as_float(v[i]);
            if (col0 + 32 > V) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (col0 + i >= V) x[i] = -kInf;
            }
            float cm = x[0];
#pragma unroll
            for (int i = 1; i < 32; ++i) cm = fmaxf(cm, x[i]);
            if (cm > m) {
                s *= ex2((m - cm) * kLog2e);
                m = cm;
            }
            const float ml2 = m * kLog2e;
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                s0 += ex2(fmaf(x[i], kLog2e, -ml2));
                s1 += ex2(fmaf(x[i + 1], kLog2e, -ml2));
            }
            s += s0 + s1;
            const unsigned d = unsigned(y - col0);
            if (d < 32u) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (d == unsigned(i)) xv = x[i];
                found = true;
            }
        }
        if (r < M) {
            part[int64_t(nt) * M + r] = make_float2(m, s);
            if (found) xy[r] = xv;
        }
    }
};

// Pass 2a: dX = c * (exp(x - lse) - onehot), rounded once to bf16, into the chunk buffer.
struct EpiDx {
    const RowRec* rec;
    const float* lse2;     // [M]: log-sum-exp of the row times log2(e); +inf for skipped rows
    const float* coef;     // [M]: gradient factor c of the row
    uint16_t* dx;          // [M, ldx] chunk buffer, column 0 = vocabulary column v0
    int64_t ldx;
    int64_t M;
    int32_t V, v0;
    int32_t v_off;         // vocabulary id of column 0 of the weight matrix
    __device__ __forceinline__ void operator()(int mt, int nt, int row, uint32_t taddr) const {
        const int64_t r = int64_t(mt) * kTileM + row;
        const bool live = r < M;
        const float l2 = live ? __ldg(lse2 + r) : kInf;
        const float cf = live ? __ldg(coef + r) : 0.f;
        const int yg = live ? load_rec(rec + r).y : -1;
        const int y = (yg >= v_off && yg - v_off < V) ? yg - v_off : -1 - kTileN;
        uint16_t* out = dx + (live ? r : 0) * ldx + nt * kTileN;
#pragma unroll 1
        for (int c = 0; c < kTileN; c += 32) {
            const int col0 = v0 + nt * kTileN + c;
            if (col0 >= V) break;
            uint32_t v[32];
            umma::tmem_ld32(taddr + c, v);
            umma::tmem_ld_wait();
            float g[32];
#pragma unroll
            for (int i = 0; i < 32; ++i)
                g[i] = cf * ex2(fmaf(__uint_as_float(v[i]), kLog2e, -l2));
            if (cf == 0.f) {     // clipped, skipped or non-finite row: exact zeros (0 * NaN is not 0)
#pragma unroll
                for (int i = 0; i < 32; ++i) g[i] = 0.f;
            }
            const unsigned d = unsigned(y - col0);
            if (d < 32u) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (d == unsigned(i)) g[i] -= cf;
            }
            if (live) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (col0 + 8 * q < V) {
                        uint4 w;
                        w.x = pack_bf16x2(g[8 * q + 0], g[8 * q + 1]);
                        w.y = pack_bf16x2(g[8 * q + 2], g[8 * q + 3]);
                        w.z = pack_bf16x2(g[8 * q + 4], g[8 * q + 5]);
                        w.w = pack_bf16x2(g[8 * q + 6], g[8 * q + 7]);
                        ptx::stg128(out + c + 8 * q, w);
                    }
                }
            }
        }
    }
};

// Pass 2b: dhidden accumulation across vocabulary chunks in fp32; the last chunk rounds to bf16.
struct EpiDh {
    float* acc;        // [M, K] fp32 running sum
    uint16_t* out;     // [M, K] bf16 result
    int64_t M;
    int32_t K;
    int32_t first, last;
    __device__ __forceinline__ void operator()(int mt, int nt, int row, uint32_t taddr) const {
        const int64_t r = int64_t(mt) * kTileM + row;
        const bool live = r < M;
#pragma unroll 1
        for (int c = 0; c < kTileN; c += 32) {
            const int col0 = nt * kTileN + c;
            if (col0 >= K) break;
            uint32_t v[32];
            umma::tmem_ld32(taddr + c, v);
            umma::tmem_ld_wait();
            if (!live) continue;
            float* a = acc + r * K + col0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (col0 + 8 * q >= K) break;
                float f[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * q + i]);
                if (!first) {
                    const float4 p0 = *reinterpret_cast<const float4*>(a + 8 * q);
                    const float4 p1 = *reinterpret_cast<const float4*>(a + 8 * q + 4);
                    f[0] += p0.x; f[1] += p0.y; f[2] += p0.z; f[3] += p0.w;
                    f[4] += p1.x; f[5] += p1.y; f[6] += p1.z; f[7] += p1.w;
                }
                if (last) {
                    uint4 w;
                    w.x = pack_bf16x2(f[0], f[1]);
                    w.y = pack_bf16x2(f[2], f[3]);
                    w.z = pack_bf16x2(f[4], f[5]);
                    w.w = pack_bf16x2(f[6], f[7]);
                    ptx::stg128(out + r * K + col0 + 8 * q, w);
                } else {
                    *reinterpret_cast<float4*>(a + 8 * q) = make_float4(f[0], f[1], f[2], f[3]);
                    *reinterpret_cast<float4*>(a + 8 * q + 4) = make_float4(f[4], f[5], f[6], f[7]);
                }
            }
        }
    }
};

// Pass 2c: one [128 x 256] block of dweight, complete (the contraction runs over all rows).
struct EpiDw {
    uint16_t* out;     // [K, V] bf16
    int32_t K, V, v0;
    __device__ __forceinline__ void operator()(int mt, int nt, int row, uint32_t taddr) const {
        const int r = mt * kTileM + row;           // row of the weight matrix
        const bool live = r < K;
#pragma unroll 1
        for (int c = 0; c < kTileN; c += 32) {
            const int col0 = v0 + nt * kTileN + c;
            if (col0 >= V) break;
            uint32_t v[32];
            umma::tmem_ld32(taddr + c, v);
            umma::tmem_ld_wait();
            if (!live) continue;
            uint16_t* o = out + int64_t(r) * V + col0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (col0 + 8 * q >= V) break;
                uint4 w;
                w.x = pack_bf16x2(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1]));
                w.y = pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3]));
                w.z = pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5]));
                w.w = pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]));
                ptx::stg128(o + 8 * q, w);
            }
        }
    }
};

// ---- per-row merge of the tile statistics and the scalar part of Eq. 1 -----------------------
__global__ void __launch_bounds__(256)
lmhead_rows_kernel(const RowRec* rec, const float2* part, const float* xy, int64_t M, int32_t n_tiles,
                   float eps_low, float eps_high, float inv_denom, float* logp, float* token_loss,
                   float* row_loss, uint8_t* row_clip, float* lse2, float* coef,
                   const float* ext_max, const float* ext_sum, const float* ext_xy, int32_t* status) {
    const int64_t r = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (r >= M) return;
    const RowRec rr = load_rec(rec + r);
    float m = -kInf, s = 0.f, x_y = 0.f;
    if (rr.y >= 0) {
        if (ext_max) {           // whole-vocabulary statistics supplied by the caller (vocabulary shards)
            m = ext_max[r];
            s = ext_sum[r];
            x_y = ext_xy[r];
        } else {
            for (int t = 0; t < n_tiles; ++t) m = fmaxf(m, part[int64_t(t) * M + r].x);
            for (int t = 0; t < n_tiles; ++t) {
                const float2 p = part[int64_t(t) * M + r];
                s += p.y * expf(p.x - m);
            }
            x_y = xy[r];
        }
    }
    // a sum of exponentials that is not positive and finite means the row's logits held a NaN or an
    // infinity (a non-finite hidden state or weight): the row is skipped and reported
    const bool finite = s > 0.f && s <= kFltMax && fabsf(m) <= kFltMax && fabsf(x_y) <= kFltMax;
    if (rr.y >= 0 && !finite) atomicOr(status, TPPO_DEV_NONFINITE);
    if (rr.y < 0 || !finite) {           // bad target or index, or non-finite logits: contributes nothing
        if (logp) logp[r] = 0.f;
        if (token_loss) token_loss[r] = 0.f;
        row_loss[r] = 0.f;
        row_clip[r] = 0;
        lse2[r] = kInf;
        coef[r] = 0.f;
        return;
    }
    const float log_sum = logf(s);
    const RowLoss rl = ppo_row(x_y - m, log_sum, rr.old_logp, rr.adv, eps_low, eps_high, inv_denom);
    if (logp) logp[r] = rl.logp;
    if (token_loss) token_loss[r] = rl.loss;
    row_loss[r] = rl.loss;
    row_clip[r] = uint8_t(rl.clip);
    lse2[r] = (m + log_sum) * kLog2e;
    coef[r] = rl.coef;
}

// Single-CTA kernels by default; the CTA-pair kernels (a third less operand traffic per FLOP, but no
// faster under the power cap that bounds this path) are selectable for comparison.
template <int AMAJ, int BMAJ, class Epi>
int launch_gemm(bool pair, const CUtensorMap& a, const CUtensorMap& b, const GemmShape& g,
                const Epi& e, int32_t* status, cudaStream_t s) {
    return pair ? launch_umma_gemm_pair<AMAJ, BMAJ>(a, b, g, e, status, s)
                : launch_umma_gemm<AMAJ, BMAJ>(a, b, g, e, status, s);
}

// Vocabulary shards: the statistics of this shard's columns for every row, to be merged by the caller
// across shards (m = max m_r, S = sum s_r exp(m_r - m), target logit = sum over shards).
__global__ void __launch_bounds__(256)
lmhead_merge_kernel(const RowRec* rec, const float2* part, const float* xy, int64_t M, int32_t n_tiles,
                    float* row_max, float* row_sum, float* row_xy) {
    const int64_t r = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (r >= M) return;
    if (load_rec(rec + r).y < 0) {       // skipped row: neutral statistics
        row_max[r] = 0.f; row_sum[r] = 0.f; row_xy[r] = 0.f;
        return;
    }
    float m = -kInf, s = 0.f;
    for (int t = 0; t < n_tiles; ++t) m = fmaxf(m, part[int64_t(t) * M + r].x);
    for (int t = 0; t < n_tiles; ++t) {
        const float2 p = part[int64_t(t) * M + r];
        s += p.y * expf(p.x - m);
    }
    row_max[r] = m;
    row_sum[r] = s;
    row_xy[r] = xy[r];
}

// Step between the two all-reduces of the vocabulary-parallel merge: bring a shard's sum of
// exponentials from its own maximum to the maximum over all shards.
__global__ void __launch_bounds__(256)
lmhead_rescale_kernel(const float* row_max, const float* row_max_all, float* row_sum, int64_t M) {
    const int64_t r = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (r >= M) return;
    const float s = row_sum[r];
    row_sum[r] = s > 0.f ? s * expf(row_max[r] - row_max_all[r]) : 0.f;
}

struct LmPlan {
    int32_t n_tiles;       // 256-column tiles of the vocabulary
    int32_t chunk_tiles;   // tiles per vocabulary chunk
};

// Chunk width: a multiple of the tile width chosen so that the three per-chunk GEMMs fill whole
// waves of 148 tiles as nearly as possible, with the chunk buffer capped at 512 MB.
LmPlan lmhead_plan(int64_t M, int32_t K, int32_t V) {
    LmPlan p;
    p.n_tiles = (V + kTileN - 1) / kTileN;
    const int64_t mt = (M + kTileM - 1) / kTileM;
    const int64_t kt256 = (K + kTileN - 1) / kTileN, kt128 = (K + kTileM - 1) / kTileM;
    const int64_t ks_k = (K + kTileK - 1) / kTileK, ks_m = (M + kTileK - 1) / kTileK;
    int64_t cap = (int64_t(512) << 20) / (int64_t(M > 0 ? M : 1) * kTileN * 2);
    if (cap < 1) cap = 1;
    if (cap > p.n_tiles) cap = p.n_tiles;
    auto waves = [](int64_t tiles) { return (tiles + kNumSms - 1) / kNumSms; };
    double best = -1.0;
    p.chunk_tiles = 1;
    for (int64_t c = 1; c <= cap; ++c) {
        const int64_t full = p.n_tiles / c, rem = p.n_tiles % c;
        auto cost = [&](int64_t w) {
            return double(waves(mt * w) * ks_k + waves(mt * kt256) * (w * (kTileN / kTileK)) +
                          waves(kt128 * w) * ks_m) + 400.0;    // + launch and accumulator traffic
        };
        const double total = double(full) * cost(c) + (rem ? cost(rem) : 0.0);
        if (best < 0.0 || total < best) { best = total; p.chunk_tiles = int32_t(c); }
    }
    return p;
}

struct LmWorkspace {
    float* row_loss; uint8_t* row_clip; RowRec* rec; float2* part; float* xy; float* lse2;
    float* coef; uint16_t* dxc; float* dhacc;
    size_t bytes;
};
LmWorkspace lmhead_carve(void* ws, int64_t M, int32_t K, int32_t V) {
    const LmPlan p = lmhead_plan(M, K, V);
    const size_t m = size_t(M > 0 ? M : 1);
    char* w = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) { char* q = w + off; off += align_up(bytes, kWsAlign); return q; };
    LmWorkspace o;
    o.row_loss = reinterpret_cast<float*>(take(m * 4));
    o.row_clip = reinterpret_cast<uint8_t*>(take(m));
    o.rec = reinterpret_cast<RowRec*>(take(m * sizeof(RowRec)));
    o.part = reinterpret_cast<float2*>(take(m * size_t(p.n_tiles) * sizeof(float2)));
    o.xy = reinterpret_cast<float*>(take(m * 4));
    o.lse2 = reinterpret_cast<float*>(take(m * 4));
    o.coef = reinterpret_cast<float*>(take(m * 4));
    o.dxc = reinterpret_cast<uint16_t*>(take(m * size_t(p.chunk_tiles) * kTileN * 2));
    o.dhacc = reinterpret_cast<float*>(take(m * size_t(K > 0 ? K : 1) * 4));
    o.bytes = off;
    return o;
}

}  // namespace

size_t lmhead_workspace_bytes(int64_t M, int32_t K, int32_t V) {
    if (M < 0 || K <= 0 || V <= 0) return kWsAlign;
    return lmhead_carve(nullptr, M, K, V).bytes;
}
}  // namespace tppo

using namespace tppo;

namespace {

enum LmMode { kLmFull = 0, kLmShardStats = 1, kLmShardGrads = 2 };

struct LmCall {
    LmMode mode;
    const void* hidden; const void* weight;
    int64_t M; int32_t K; int32_t V;          // V: columns of `weight` (the shard width)
    int32_t v_off; int32_t V_total;           // vocabulary id of column 0, size of the whole vocabulary
    const int32_t* targets; const int32_t* aux_idx; const float* old_logp; const float* adv;
    int64_t aux_len; float eps_low, eps_high, denom;
    const float* in_max; const float* in_sum; const float* in_xy;    // kLmShardGrads: whole-vocabulary statistics
    float* out_max; float* out_sum; float* out_xy;                   // kLmShardStats: this shard's statistics
    float* logp; float* token_loss; float* loss; int32_t* stats;
    void* dhidden; void* dweight; int32_t chunk_tiles;
    void* workspace; size_t workspace_bytes; void* stream;
};

int lmhead_run(const LmCall& c) {
    const int64_t M = c.M;
    const int32_t K = c.K, V = c.V;
    if (M < 0 || K <= 0 || V <= 0 || c.aux_len < 0 || M >= (int64_t(1) << 31) - kTileM)
        return TPPO_ERR_INVALID_ARG;
    if (c.v_off < 0 || c.V_total < V || c.v_off > c.V_total - V) return TPPO_ERR_INVALID_ARG;
    if (!c.stats) return TPPO_ERR_INVALID_ARG;
    if (c.mode != kLmShardStats && !c.loss) return TPPO_ERR_INVALID_ARG;
    if (M > 0 && (!c.hidden || !c.weight || !c.targets)) return TPPO_ERR_INVALID_ARG;
    if (M > 0 && c.mode != kLmShardStats && (!c.old_logp || !c.adv)) return TPPO_ERR_INVALID_ARG;
    if (M > 0 && c.mode == kLmShardStats && (!c.out_max || !c.out_sum || !c.out_xy))
        return TPPO_ERR_INVALID_ARG;
    if (M > 0 && c.mode == kLmShardGrads && (!c.in_max || !c.in_sum || !c.in_xy))
        return TPPO_ERR_INVALID_ARG;
    if (!(c.eps_low >= 0.f) || !(c.eps_high >= 0.f) || c.chunk_tiles < 0) return TPPO_ERR_INVALID_ARG;
    // TMA row strides and the 16-byte vector stores need K and V to be multiples of 8 bf16.
    if (K % 8 != 0 || V % 8 != 0) return TPPO_ERR_UNSUPPORTED;
    if (!aligned(c.hidden, 16) || !aligned(c.weight, 16) || (c.dhidden && !aligned(c.dhidden, 16)) ||
        (c.dweight && !aligned(c.dweight, 16)))
        return TPPO_ERR_INVALID_ARG;
    if (!c.workspace || !aligned(c.workspace, kWsAlign) ||
        c.workspace_bytes < lmhead_workspace_bytes(M, K, V))
        return TPPO_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(c.stream);
    const LmWorkspace w = lmhead_carve(c.workspace, M, K, V);
    LmPlan plan = lmhead_plan(M, K, V);
    const int64_t ldx = int64_t(plan.chunk_tiles) * kTileN;     // row stride of the chunk buffer
    const bool pair = (c.chunk_tiles & 0x10000) != 0;           // bit 16: CTA-pair kernels
    const int32_t chunk_tiles = c.chunk_tiles & 0xffff;
    if (chunk_tiles > 0 && chunk_tiles < plan.chunk_tiles) plan.chunk_tiles = chunk_tiles;
    int32_t* stats = c.stats;

    // Targets are validated against the whole vocabulary; columns are local to the shard.
    PolicyArgs a{};
    a.logits = nullptr; a.R = M; a.V = c.V_total; a.ld = c.V_total; a.targets = c.targets;
    a.rows = nullptr; a.n_sel = nullptr; a.n_max = M; a.aux_idx = c.aux_idx;
    a.old_logp = c.old_logp; a.adv = c.adv; a.aux_len = c.aux_len; a.eps_low = c.eps_low;
    a.eps_high = c.eps_high; a.denom = c.denom; a.logp = c.logp; a.token_loss = c.token_loss;
    a.loss = c.loss; a.stats = stats; a.dlogits = nullptr; a.mode = TPPO_DLOGITS_NONE;
    a.row_loss = w.row_loss; a.row_clip = w.row_clip; a.row_flag = nullptr; a.rec = w.rec;

    TPPO_CUDA_CHECK(cudaMemsetAsync(stats, 0, 4 * sizeof(int32_t), s));
    if (M == 0) return c.mode == kLmShardStats ? TPPO_OK : launch_policy_finish(a, s);
    int rc = launch_policy_prepare(a, s);
    if (rc != TPPO_OK) return rc;

    const int32_t mt = int32_t((M + kTileM - 1) / kTileM);
    const int32_t ks_k = (K + kTileK - 1) / kTileK;
    const int32_t ks_m = int32_t((M + kTileK - 1) / kTileK);
    CUtensorMap map_h128, map_h64, map_w64, map_w256;
    if (!make_bf16_tensor_map(&map_h128, c.hidden, uint64_t(M), uint64_t(K), uint64_t(K), 128) ||
        !make_bf16_tensor_map(&map_h64, c.hidden, uint64_t(M), uint64_t(K), uint64_t(K), 64) ||
        !make_bf16_tensor_map(&map_w64, c.weight, uint64_t(K), uint64_t(V), uint64_t(V), 64) ||
        !make_bf16_tensor_map(&map_w256, c.weight, uint64_t(K), uint64_t(V), uint64_t(V),
                              pair ? 128 : 256))     // K-major B box: 128 rows per CTA of a pair
        return TPPO_ERR_CUDA;

    // pass 1: statistics over the columns of this weight matrix
    if (c.mode != kLmShardGrads) {
        TPPO_CUDA_CHECK(cudaMemsetAsync(w.xy, 0, size_t(M) * 4, s));
        const GemmShape g{mt, plan.n_tiles, ks_k, 0, 0, 0, 0, 16};
        const EpiStats e{w.rec, w.part, w.xy, M, V, c.v_off};
        rc = launch_gemm<0, 1>(pair, map_h128, map_w64, g, e, stats + 3, s);
        if (rc != TPPO_OK) return rc;
    }
    if (c.mode == kLmShardStats) {
        lmhead_merge_kernel<<<unsigned((M + 255) / 256), 256, 0, s>>>(
            w.rec, w.part, w.xy, M, plan.n_tiles, c.out_max, c.out_sum, c.out_xy);
        TPPO_CUDA_CHECK(cudaGetLastError());
        return TPPO_OK;
    }
    const float inv_denom = c.denom > 0.f ? 1.f / c.denom : 1.f / float(M);
    lmhead_rows_kernel<<<unsigned((M + 255) / 256), 256, 0, s>>>(
        w.rec, w.part, w.xy, M, plan.n_tiles, c.eps_low, c.eps_high, inv_denom, c.logp, c.token_loss,
        w.row_loss, w.row_clip, w.lse2, w.coef, c.in_max, c.in_sum, c.in_xy, stats + 3);
    TPPO_CUDA_CHECK(cudaGetLastError());
    rc = launch_policy_finish(a, s);
    if (rc != TPPO_OK) return rc;
    if (!c.dhidden && !c.dweight) return TPPO_OK;

    // pass 2: gradients, one vocabulary chunk at a time
    const int32_t chunk_cols = plan.chunk_tiles * kTileN;
    const int32_t n_chunks = (plan.n_tiles + plan.chunk_tiles - 1) / plan.chunk_tiles;
    for (int32_t ci = 0; ci < n_chunks; ++ci) {
        const int32_t v0 = ci * chunk_cols;
        const int32_t width = V - v0 < chunk_cols ? V - v0 : chunk_cols;
        const int32_t ct = (width + kTileN - 1) / kTileN;
        CUtensorMap map_dx128, map_dx64;
        if (!make_bf16_tensor_map(&map_dx128, w.dxc, uint64_t(M), uint64_t(width), uint64_t(ldx), 128) ||
            !make_bf16_tensor_map(&map_dx64, w.dxc, uint64_t(M), uint64_t(width), uint64_t(ldx), 64))
            return TPPO_ERR_CUDA;
        {
            const GemmShape g{mt, ct, ks_k, 0, 0, v0, 0, 16};
            const EpiDx e{w.rec, w.lse2, w.coef, w.dxc, ldx, M, V, v0, c.v_off};
            rc = launch_gemm<0, 1>(pair, map_h128, map_w64, g, e, stats + 3, s);
            if (rc != TPPO_OK) return rc;
        }
        if (c.dhidden) {
            const GemmShape g{mt, (K + kTileN - 1) / kTileN, (width + kTileK - 1) / kTileK,
                              0, 0, 0, v0, 16};
            const EpiDh e{w.dhacc, static_cast<uint16_t*>(c.dhidden), M, K, ci == 0,
                          ci == n_chunks - 1};
            rc = launch_gemm<0, 0>(pair, map_dx128, map_w256, g, e, stats + 3, s);
            if (rc != TPPO_OK) return rc;
        }
        if (c.dweight) {
            const GemmShape g{(K + kTileM - 1) / kTileM, ct, ks_m, 0, 0, 0, 0, 16};
            const EpiDw e{static_cast<uint16_t*>(c.dweight), K, V, v0};
            rc = launch_gemm<1, 1>(pair, map_h64, map_dx64, g, e, stats + 3, s);
            if (rc != TPPO_OK) return rc;
        }
    }
    return TPPO_OK;
}

}  // namespace

TPPO_API int tppo_lmhead_logprob_fwd_bwd(const void* hidden, const void* weight, int64_t M, int32_t K,
                                         int32_t V, const int32_t* targets, const int32_t* aux_idx,
                                         const float* old_logp, const float* adv, int64_t aux_len,
                                         float eps_low, float eps_high, float denom, float* logp,
                                         float* token_loss, float* loss, int32_t* stats,
                                         void* dhidden, void* dweight, int32_t chunk_tiles,
                                         void* workspace, size_t workspace_bytes, void* stream) {
    LmCall c{};
    c.mode = kLmFull; c.hidden = hidden; c.weight = weight; c.M = M; c.K = K; c.V = V;
    c.v_off = 0; c.V_total = V; c.targets = targets; c.aux_idx = aux_idx; c.old_logp = old_logp;
    c.adv = adv; c.aux_len = aux_len; c.eps_low = eps_low; c.eps_high = eps_high; c.denom = denom;
    c.logp = logp; c.token_loss = token_loss; c.loss = loss; c.stats = stats; c.dhidden = dhidden;
    c.dweight = dweight; c.chunk_tiles = chunk_tiles; c.workspace = workspace;
    c.workspace_bytes = workspace_bytes; c.stream = stream;
    return lmhead_run(c);
}

TPPO_API int tppo_lmhead_shard_stats(const void* hidden, const void* weight_shard, int64_t M, int32_t K,
                                     int32_t V_shard, int32_t v_offset, int32_t V_total,
                                     const int32_t* targets, float* row_max, float* row_sumexp,
                                     float* row_target_logit, int32_t* stats, int32_t chunk_tiles,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    LmCall c{};
    c.mode = kLmShardStats; c.hidden = hidden; c.weight = weight_shard; c.M = M; c.K = K;
    c.V = V_shard; c.v_off = v_offset; c.V_total = V_total; c.targets = targets;
    c.aux_len = M;      // no per-token scalars are read here: every row with a valid target counts
    c.out_max = row_max; c.out_sum = row_sumexp; c.out_xy = row_target_logit; c.stats = stats;
    c.chunk_tiles = chunk_tiles; c.workspace = workspace; c.workspace_bytes = workspace_bytes;
    c.stream = stream;
    return lmhead_run(c);
}

TPPO_API int tppo_lmhead_shard_fwd_bwd(const void* hidden, const void* weight_shard, int64_t M,
                                       int32_t K, int32_t V_shard, int32_t v_offset, int32_t V_total,
                                       const int32_t* targets, const int32_t* aux_idx,
                                       const float* old_logp, const float* adv, int64_t aux_len,
                                       float eps_low, float eps_high, float denom,
                                       const float* row_max, const float* row_sumexp,
                                       const float* row_target_logit, float* logp, float* token_loss,
                                       float* loss, int32_t* stats, void* dhidden_partial,
                                       void* dweight_shard, int32_t chunk_tiles, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    LmCall c{};
    c.mode = kLmShardGrads; c.hidden = hidden; c.weight = weight_shard; c.M = M; c.K = K;
    c.V = V_shard; c.v_off = v_offset; c.V_total = V_total; c.targets = targets; c.aux_idx = aux_idx;
    c.old_logp = old_logp; c.adv = adv; c.aux_len = aux_len; c.eps_low = eps_low;
    c.eps_high = eps_high; c.denom = denom; c.in_max = row_max; c.in_sum = row_sumexp;
    c.in_xy = row_target_logit; c.logp = logp; c.token_loss = token_loss; c.loss = loss;
    c.stats = stats; c.dhidden = dhidden_partial; c.dweight = dweight_shard;
    c.chunk_tiles = chunk_tiles; c.workspace = workspace; c.workspace_bytes = workspace_bytes;
    c.stream = stream;
    return lmhead_run(c);
}

TPPO_API int tppo_lmhead_shard_rescale(const float* row_max, const float* row_max_all,
                                       float* row_sumexp, int64_t M, void* stream) {
    if (M < 0) return TPPO_ERR_INVALID_ARG;
    if (M == 0) return TPPO_OK;
    if (!row_max || !row_max_all || !row_sumexp) return TPPO_ERR_INVALID_ARG;
    lmhead_rescale_kernel<<<unsigned((M + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        row_max, row_max_all, row_sumexp, M);
    TPPO_CUDA_CHECK(cudaGetLastError());
    return TPPO_OK;
}
