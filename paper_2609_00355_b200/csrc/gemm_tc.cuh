// Interface of the tcgen05 weight-streaming GEMM (definitions in gemm_tc.cu).
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace glance {

constexpr int kTopkTileCap = 16;     // candidate keys a (tile, row) pair may emit (>= the largest k)

struct TcGemmArgs {
    int Nout, K, R, S;          // W [Nout][K], X [R][K]; S = split-K factor (modes 0, 3, 4; 1 otherwise)
    int x_lo_row;               // > 0: X is two-term (hi + lo, both bf16); the lo plane starts at this row of the X map
    // mode 0: fp32 planes Y[split][r][f]; mode 2: optional fp32 logits Y[r][f] (may be nullptr)
    float *Y;
    int ldy;
    size_t split_stride;
    // mode 1 (SwiGLU): W holds F gate rows then F up rows; act[r][f] = silu(gate) * up
    bf16 *act, *act_lo;         // act_lo: second term of the two-term output, or nullptr
    int F;
    // mode 2 (arg-max over f): keys[r] packed (value, id) merged with atomicMax; the last CTA writes argmax[r]
    unsigned long long *keys;
    int32_t *argmax;
    int32_t *counter;
    int32_t *status;
    // mode 2, sampling: sample_pos[r] = position of row r (the draw is for position + 1), or nullptr for the plain
    // arg-max; values are scaled by sample_inv_t and perturbed by the Gumbel field of (sample_seed, position, id)
    const int32_t *sample_pos;
    unsigned long long sample_seed;
    float sample_inv_t;
    // mode 2, root-entropy log: rows r with r % ent_N == 0 are round roots; every tile leaves (max, sum exp, sum exp *
    // logit) of its 128 features in ent_part [tiles][ent_batch][3] and the last CTA writes the entropy (nats) of
    // sequence r / ent_N to ent_out; ent_out == nullptr: off
    float *ent_part, *ent_out;
    int ent_N, ent_batch;
    // mode 5 (top-k of the draft block): rows r with r % tk_B != 0 leave, per 128-feature tile, (max, sum exp) in
    // tk_ml [tiles][R][2], up to kTopkTileCap packed (value, id) keys in tk_cand [tiles][R][kTopkTileCap] and their
    // number in tk_cnt [tiles][R]; tk_thr [R][kTopkTileCap] holds, per row, the order-preserving images of tk_k running
    // maxima (class c = tiles with index % tk_k == c; 0 = empty; raised with atomicMax, re-armed by the merge kernel):
    // their minimum is a bound that at least tk_k entries of the row reach
    int tk_k, tk_B;
    uint32_t *tk_thr;
    float *tk_ml;
    int32_t *tk_cnt;
    unsigned long long *tk_cand;
    // row scales (modes 0, 1, 2, 4, 5): row r is multiplied by rsqrt(sum_i ssq[i*ssq_stride + r] / K + eps); nullptr = 1
    const float *ssq;
    int n_ssq, ssq_stride;
    float eps;
    // mode 3 (residual): x[r][f] += result; xb = bf16(x * gain[f]); ssq_out[tile][r] = sum over the tile of x^2
    float *x;
    const bf16 *gain;
    bf16 *xb, *xb_lo, *hidden_out;
    float *ssq_out;
    // mode 4 (rotary + K/V write): features are q heads, then k heads, then v heads, head_dim wide
    bf16 *q, *q_lo;      // mode 4: rotated queries, and the second term of their two-term form (or nullptr)
    bf16 *pool_layer;
    const long long *kvrow;      // [R] element offset of the row's K slot for kv head 0 inside the layer, -1 = none
    size_t v_off, head_stride;
    const float *rope_cos, *rope_sin;   // [R][head_dim/2]
    int Hq, Hkv, head_dim, Rq;
    unsigned long long *trace;   // test hook: 16 phase timestamps (ns) of CTA (0,0,0), or nullptr
    // test hook for the bounded waits: every wait of the launch gives up after wait_limit_ns (0 = the regular limit),
    // and the producer never fills the ring slot of k-step stall_kstep1 - 1 (0 = none), so the consumer's wait on it
    // runs out
    unsigned long long wait_limit_ns;
    int stall_kstep1;
    // filled by launch_gemm_tc
    int np, stages, rows_fastest;
    uint32_t tmem_cols;
};

// 2-D bf16 tensor map {inner = K, rows}, box {64, box_rows}, 128-byte swizzle.  Host call, no device work.
bool tc_make_map(CUtensorMap *map, const void *base, uint64_t inner, uint64_t rows, uint32_t box_rows);
// activation rows per CTA, padded to the UMMA N granularity (box_rows of the X map)
int tc_row_pad(int R);
// mode: 0 fp32 planes, 1 SwiGLU, 2 arg-max, 3 cluster split-K + residual, 4 cluster split-K + rotary/KV write,
// 5 per-tile top-k candidates + log-sum-exp shares.
// map_w box_rows must be 128 (64 in mode 1), map_x box_rows tc_row_pad(R).
cudaError_t launch_gemm_tc(int mode, TcGemmArgs a, const CUtensorMap &map_w, const CUtensorMap &map_x, cudaStream_t st);

}  // namespace glance
