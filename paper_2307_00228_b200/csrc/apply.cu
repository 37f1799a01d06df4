// Apply: the dense transform of a layer.  This file holds the weight preparation kernel and
// the fp32 CUDA-core GEMM (exact fp32 products, fp32 accumulation) with the routed epilogue.
#include "common.cuh"

namespace {

__device__ __forceinline__ float act_apply(float x, int act) {
  if (act == IT_ACT_RELU) return fmaxf(x, 0.f);
  if (act == IT_ACT_ELU) return it_elu(x);
  return x;
}

__device__ __forceinline__ float load_as_float(const void *p, int64_t i, int is_bf16) {
  return is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(p)[i])
                 : reinterpret_cast<const float *>(p)[i];
}

// ----------------------------------------------------------------------------- weight prep
struct PrepParams {
  int kind, in_dim, out_dim, heads, w_is_bf16;
  int k_rows;   // rows of W that a plain copy takes (SAGE: 2 in_dim + edge_dim; dense / GCN: in_dim (+ edge_dim))
  const void *W;
  const float *att_src, *att_dst;
  float *B;
};

__global__ void prep_weights_kernel(PrepParams p) {
  const int fi = p.in_dim, fo = p.out_dim;
  if (p.kind == IT_PREP_SAGE || p.kind == IT_PREP_DENSE) {
    int64_t total = (int64_t)p.k_rows * fo;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x)
      p.B[i] = load_as_float(p.W, i, p.w_is_bf16);
  } else if (p.kind == IT_PREP_SAGE_REORDER) {
    // B[k, c] = W[k, c] (self), B[k, fo + c] = W[fi + k, c] (neighbour)
    int64_t total = (int64_t)fi * 2 * fo;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      int k = (int)(i / (2 * fo)), c = (int)(i % (2 * fo));
      p.B[i] = c < fo ? load_as_float(p.W, (int64_t)k * fo + c, p.w_is_bf16)
                      : load_as_float(p.W, (int64_t)(fi + k) * fo + (c - fo), p.w_is_bf16);
    }
  } else {
    // GAT: B = [W | W a_src | W a_dst]; column fo + h is sum_c W[k, h*D + c] * a_src[h, c]
    const int nb = fo + 2 * p.heads, D = fo / p.heads;
    int64_t total = (int64_t)fi * nb;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
      int k = (int)(i / nb), c = (int)(i % nb);
      if (c < fo) {
        p.B[i] = load_as_float(p.W, (int64_t)k * fo + c, p.w_is_bf16);
      } else {
        int h = (c - fo) % p.heads;
        const float *att = (c - fo) < p.heads ? p.att_src : p.att_dst;
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
          acc += (double)load_as_float(p.W, (int64_t)k * fo + h * D + d, p.w_is_bf16) * (double)att[h * D + d];
        p.B[i] = (float)acc;
      }
    }
  }
}

// ----------------------------------------------------------------------------- fp32 GEMM
constexpr int BM = 128, BN = 64, BK = 16, GEMM_THREADS = 256;

struct GemmParams {
  int64_t M;
  const void *X1; int K1;
  const void *X2; int K2;
  const float *B; int NB;
  int n0; void *out0; int out0_bf16; const float *bias0; int act0;
  int n1; void *out1; int out1_bf16;
  float *out2;
};

template <typename T>
__global__ void __launch_bounds__(GEMM_THREADS) gemm_fp32_kernel(GemmParams p) {
  __shared__ float Xs[BK][BM + 4];
  __shared__ float Bs[BK][BN];
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;  // 16 x 16 threads, each 8 rows x 4 cols
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int c0 = blockIdx.y * BN;
  const int K = p.K1 + p.K2;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int lr = tid / 2, lk = (tid % 2) * 8;  // X tile: row lr, 8 consecutive k starting at lk
  for (int k0 = 0; k0 < K; k0 += BK) {
    {
      const int64_t m = m0 + lr;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int k = k0 + lk + q;
        float x = 0.f;
        if (m < p.M && k < K) {
          if (k < p.K1) x = (float)reinterpret_cast<const T *>(p.X1)[m * p.K1 + k];
          else x = (float)reinterpret_cast<const T *>(p.X2)[m * p.K2 + (k - p.K1)];
        }
        Xs[lk + q][lr] = x;
      }
      const int br = tid / 16, bc = (tid % 16) * 4;  // B tile: row br, 4 consecutive columns
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int k = k0 + br, c = c0 + bc + q;
        Bs[br][bc + q] = (k < K && c < p.NB) ? p.B[(int64_t)k * p.NB + c] : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[8], b[4];
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = Xs[kk][ty * 8 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  const int n01 = p.n0 + p.n1, n2 = p.NB - n01;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t m = m0 + ty * 8 + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + tx * 4 + j;
      if (c >= p.NB) continue;
      float v = acc[i][j];
      if (c < p.n0) {
        if (p.bias0) v += p.bias0[c];
        v = act_apply(v, p.act0);
        if (p.out0_bf16) reinterpret_cast<__nv_bfloat16 *>(p.out0)[m * p.n0 + c] = __float2bfloat16_rn(v);
        else reinterpret_cast<float *>(p.out0)[m * p.n0 + c] = v;
      } else if (c < n01) {
        if (p.out1_bf16) reinterpret_cast<__nv_bfloat16 *>(p.out1)[m * p.n1 + (c - p.n0)] = __float2bfloat16_rn(v);
        else reinterpret_cast<float *>(p.out1)[m * p.n1 + (c - p.n0)] = v;
      } else {
        p.out2[m * n2 + (c - n01)] = v;
      }
    }
  }
}

}  // namespace

it_status it_launch_prep_weights(it_prep_kind kind, const it_layer_desc *L, int K, float *B, cudaStream_t st) {
  PrepParams p;
  p.k_rows = K;
  p.kind = kind; p.in_dim = L->in_dim; p.out_dim = L->out_dim; p.heads = L->heads;
  p.w_is_bf16 = L->weight_dtype == IT_BF16; p.W = L->W; p.att_src = L->att_src; p.att_dst = L->att_dst; p.B = B;
  IT_LAUNCH(IT_K_PREP, 0, 0, st, prep_weights_kernel<<<64, 256, 0, st>>>(p));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}

it_status it_launch_gemm(const it_gemm_args &a, cudaStream_t st) {
  if (a.M == 0) return IT_OK;
  GemmParams p;
  p.M = a.M; p.X1 = a.X1; p.K1 = a.K1; p.X2 = a.X2; p.K2 = a.X2 ? a.K2 : 0; p.B = a.B; p.NB = a.NB;
  p.n0 = a.n0; p.out0 = a.out0; p.out0_bf16 = a.dt0 == IT_BF16; p.bias0 = a.bias0; p.act0 = a.act0;
  p.n1 = a.n1; p.out1 = a.out1; p.out1_bf16 = a.dt1 == IT_BF16; p.out2 = (float *)a.out2;
  dim3 grid((unsigned)((a.M + BM - 1) / BM), (unsigned)((a.NB + BN - 1) / BN));
  // algorithmic traffic: every operand and every result once; flops 2*M*K*N
  const double xs = a.x_dtype == IT_F32 ? 4.0 : 2.0;
  const double K = (double)(p.K1 + p.K2);
  const double bytes = (double)a.M * (K * xs + a.n0 * (a.dt0 == IT_F32 ? 4.0 : 2.0) + a.n1 * (a.dt1 == IT_F32 ? 4.0 : 2.0) +
                                     (a.NB - a.n0 - a.n1) * 4.0) + K * a.NB * xs;
  const double flops = 2.0 * (double)a.M * K * a.NB;
  if (a.x_dtype == IT_F32) IT_LAUNCH(IT_K_GEMM_FP32, bytes, flops, st, gemm_fp32_kernel<float><<<grid, GEMM_THREADS, 0, st>>>(p));
  else IT_LAUNCH(IT_K_GEMM_FP32, bytes, flops, st, gemm_fp32_kernel<__nv_bfloat16><<<grid, GEMM_THREADS, 0, st>>>(p));
  IT_CUDA_TRY(cudaGetLastError());
  return IT_OK;
}
