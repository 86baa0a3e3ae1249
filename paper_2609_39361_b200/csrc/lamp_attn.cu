// LampAttention forward for B200 (sm_100a): kernels and the C ABI of include/lamp_attn.h.
#include "lamp_attn.h"

#include <math.h>
#include <string.h>

#include "lamp_common.cuh"
#include "lamp_tile.cuh"

namespace lamp {

__device__ DeviceStats g_stats;
__constant__ uint32_t c_lut8[256];   // fp32 bits of the 8-bit exponential | its byte

// ---------------------------------------------------------------------------------------
// Reference-structure kernel: CUDA cores only.  One CTA = 128 query rows of one (b, h),
// four warps, one group of 32 rows each; key tiles visited in ascending order (the flags
// depend on the history of the running maxima, so the key dimension is never split).
template <int D, bool DUMP>
__global__ void __launch_bounds__(128, 1) lamp_fwd_simt(const __grid_constant__ KernelParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* qsT = reinterpret_cast<float*>(smem_raw);                    // [D][128] q * scale
  float* kf = qsT + D * kBM;                                          // [D][kKfStride]
  __nv_bfloat16* vs = reinterpret_cast<__nv_bfloat16*>(kf + D * kKfStride);  // [64][D]
  float* es_all = reinterpret_cast<float*>(vs + kTK * D);             // [4][64][32]
  float* os = es_all + 4 * kTK * kBQ;                                 // [128][D]
  float* rowbuf = os + kBM * D;                                       // [128]
  uint32_t* lut = reinterpret_cast<uint32_t*>(rowbuf + kBM);          // [256]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int qa = lane >> 2, th_own = lane & 3;
  const int ntq = P.seqlen / kBM;
  const int qt = ntq - 1 - blockIdx.x;            // long (late) query tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int hk = h / (P.heads_q / P.heads_kv);
  const int m0 = qt * kBM;
  const int j0 = m0 + warp * kBQ;

  const __nv_bfloat16* qg = P.q + b * P.qs[0] + h * P.qs[1] + (int64_t)m0 * P.qs[2];
  const __nv_bfloat16* kg = P.k + b * P.ks[0] + hk * P.ks[1];
  const __nv_bfloat16* vg = P.v + b * P.vs[0] + hk * P.vs[1];

  for (int i = tid; i < 256; i += 128) lut[i] = c_lut8[i];
  for (int c = tid; c < kBM * D / 8; c += 128) {
    const int row = c / (D / 8), k0 = (c % (D / 8)) * 8;
    const uint4 raw = *reinterpret_cast<const uint4*>(qg + (int64_t)row * P.qs[2] + k0);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const uint32_t w = (&raw.x)[e >> 1];
      const float f = __uint_as_float((e & 1) ? (w & 0xffff0000u) : (w << 16));
      qsT[(k0 + e) * kBM + row] = __fmul_rn(f, P.scale);
    }
  }
  for (int c = tid; c < kBM * D; c += 128) os[c] = 0.0f;

  RowState st;
#pragma unroll
  for (int a = 0; a < 4; ++a) { st.mu[a] = -INFINITY; st.om[a] = 0.0f; }
  WarpCounters wc;
  memset(&wc, 0, sizeof(wc));

  int t_begin = 0, t_end = P.seqlen / kTK;
  if (P.causal) t_end = min(t_end, (m0 + kBM - 1) / kTK + 1);
  if (P.window > 0) t_begin = max(0, m0 - P.window + 1) / kTK;
  const int ntk = P.seqlen / kTK;
  const bool dump_rows = DUMP && b == P.dbg_batch && h == P.dbg_head;
  float* es = es_all + warp * kTK * kBQ;

  for (int t = t_begin; t < t_end; ++t) {
    const int i0 = t * kTK;
    __syncthreads();   // previous tile fully consumed
    for (int c = tid; c < kTK * D / 8; c += 128) {
      const int key = c / (D / 8), k0 = (c % (D / 8)) * 8;
      const uint4 raw = *reinterpret_cast<const uint4*>(kg + (int64_t)(i0 + key) * P.ks[2] + k0);
      const uint4 rawv = *reinterpret_cast<const uint4*>(vg + (int64_t)(i0 + key) * P.vs[2] + k0);
      *reinterpret_cast<uint4*>(vs + key * D + k0) = rawv;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t w = (&raw.x)[e >> 1];
        kf[(k0 + e) * kKfStride + kf_pos(key)] =
            __uint_as_float((e & 1) ? (w & 0xffff0000u) : (w << 16));
      }
    }
    __syncthreads();

    TileGeom g;
    g.i0 = i0; g.j0 = j0; g.causal = P.causal; g.window = P.window;
    const bool any = (!P.causal || i0 <= j0 + 31) && (P.window == 0 || j0 - (i0 + 63) < P.window);
    g.full = (!P.causal || i0 + 63 <= j0) && (P.window == 0 || (j0 + 31) - i0 < P.window);
    float lam[4] = {1.0f, 1.0f, 1.0f, 1.0f};
    uint32_t flag = 0;
    unsigned long long cks[2] = {0ull, 0ull};
    if (any) {
      const int dump0 = dump_rows ? j0 : -1;
      const __nv_bfloat16* qrow = qg + (int64_t)(warp * kBQ + 4 * qa) * P.qs[2];
      if (g.full)
        flag = lamp_tile<D, true, DUMP>(P, g, qsT + warp * kBQ + 4 * qa, kBM, kf, qrow, lut, es,
                                        st, lam, wc, cks, dump0);
      else
        flag = lamp_tile<D, false, DUMP>(P, g, qsT + warp * kBQ + 4 * qa, kBM, kf, qrow, lut, es,
                                         st, lam, wc, cks, dump0);
    }
    const int64_t gt = (((int64_t)b * P.heads_q + h) * (P.seqlen / kBQ) + (j0 / kBQ)) * ntk + t;
    if (lane == 0 && P.flag_mask) P.flag_mask[gt] = (uint8_t)flag;
    if (DUMP && P.dbg_checksums) {
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) {
        cks[0] += __shfl_xor_sync(kFull, cks[0], s);
        cks[1] += __shfl_xor_sync(kFull, cks[1], s);
      }
      if (lane == 0) { P.dbg_checksums[2 * gt] = cks[0]; P.dbg_checksums[2 * gt + 1] = cks[1]; }
    }
    if (!any) continue;   // warp-uniform; the __syncthreads above are outside this branch

    // O <- diag(lambda) O + E^T V on the CUDA cores (fp32): lane = 4 output columns
    if (th_own == 0) {
#pragma unroll
      for (int a = 0; a < 4; ++a) rowbuf[warp * kBQ + 4 * qa + a] = lam[a];
    }
    __syncwarp();
    for (int jq = 0; jq < kBQ; jq += 4) {
      float o[4][D / 32];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < D / 32; ++c)
          o[a][c] = rowbuf[warp * kBQ + jq + a] * os[(warp * kBQ + jq + a) * D + lane + 32 * c];
      for (int i = 0; i < kTK; ++i) {
        const float4 e4 = *reinterpret_cast<const float4*>(es + i * kBQ + jq);
        if (e4.x == 0.0f && e4.y == 0.0f && e4.z == 0.0f && e4.w == 0.0f) continue;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          const float vv = __bfloat162float(vs[i * D + lane + 32 * c]);
          o[0][c] = fmaf(e4.x, vv, o[0][c]);
          o[1][c] = fmaf(e4.y, vv, o[1][c]);
          o[2][c] = fmaf(e4.z, vv, o[2][c]);
          o[3][c] = fmaf(e4.w, vv, o[3][c]);
        }
      }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < D / 32; ++c) os[(warp * kBQ + jq + a) * D + lane + 32 * c] = o[a][c];
    }
    __syncwarp();
  }

  // ---- epilogue: O / omega, lse = mu + ln(omega) ------------------------------------------
  if (th_own == 0) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      rowbuf[warp * kBQ + 4 * qa + a] = st.om[a];
      if (P.lse)
        P.lse[((int64_t)b * P.heads_q + h) * P.seqlen + j0 + 4 * qa + a] =
            (float)((double)st.mu[a] + log((double)st.om[a]));
    }
  }
  __syncwarp();
  for (int j = 0; j < kBQ; ++j) {
    const float den = rowbuf[warp * kBQ + j];
    const int64_t orow = b * P.os[0] + h * P.os[1] + (int64_t)(j0 + j) * P.os[2];
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      const float val = os[(warp * kBQ + j) * D + lane + 32 * c] / den;
      if (P.flags & LAMP_OUT_FP32) reinterpret_cast<float*>(P.out)[orow + lane + 32 * c] = val;
      else reinterpret_cast<__nv_bfloat16*>(P.out)[orow + lane + 32 * c] = __float2bfloat16(val);
    }
  }

  // ---- counters --------------------------------------------------------------------------
  const unsigned sat8 = __reduce_add_sync(kFull, wc.sat8);
  const unsigned sat16 = __reduce_add_sync(kFull, wc.sat16);
  const unsigned gt1 = __reduce_add_sync(kFull, wc.gt1);
  if (lane == 0) {
    atomicAdd(&g_stats.v[0], wc.active);
    atomicAdd(&g_stats.v[1], wc.s1);
    atomicAdd(&g_stats.v[2], wc.s2);
#pragma unroll
    for (int i = 0; i < 5; ++i) atomicAdd(&g_stats.v[3 + i], wc.hist[i]);
    atomicAdd(&g_stats.v[8], (unsigned long long)sat8);
    atomicAdd(&g_stats.v[9], (unsigned long long)sat16);
    atomicAdd(&g_stats.v[10], (unsigned long long)gt1);
    atomicAdd(&g_stats.v[11], wc.bigrow);
  }
}

template <int D>
constexpr size_t simt_smem_bytes() {
  return sizeof(float) * (D * kBM + D * kKfStride + 4 * kTK * kBQ + kBM * D + kBM) +
         sizeof(__nv_bfloat16) * kTK * D + 256 * sizeof(uint32_t);
}

// ---------------------------------------------------------------------------------------
// Host side: the exponential table, argument checks, launch.

// Round v in [0, 1] to the 8-bit exponential grid (value = 2^(E-31)(1 + M/8), E >= 1;
// 2^-30 M/8 for E = 0; 0xF8 = 1.0), nearest-even; returns the byte and the grid value.
static uint32_t exp8_entry(double s) {
  const double v = exp(-s);
  int e;
  frexp(v, &e);
  int ex = e - 1;
  if (v == 0.0 || ex < -30) ex = -30;
  const double q = ldexp(1.0, ex - 3);
  const double r = nearbyint(v / q) * q;
  if (r == 0.0) return 0u;
  uint32_t byte;
  if (r < ldexp(1.0, -30)) byte = (uint32_t)(r / ldexp(1.0, -33));
  else {
    int e2;
    const double m = frexp(r, &e2);
    byte = (uint32_t)(((e2 - 1 + 31) << 3) | (int)((m * 2.0 - 1.0) * 8.0));
  }
  const float rf = (float)r;
  uint32_t bits;
  memcpy(&bits, &rf, 4);
  return (bits & 0xffffff00u) | byte;
}

static thread_local int t_last_cuda = 0;
static int cuda_fail(cudaError_t e) {
  t_last_cuda = (int)e;
  return LAMP_ERR_CUDA;
}

struct DeviceInit {
  bool ready[64] = {};
};
static DeviceInit g_init;

static int ensure_device(int* dev_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  *dev_out = dev;
  if (dev < 64 && g_init.ready[dev]) return LAMP_OK;
  cudaDeviceProp prop;
  e = cudaGetDeviceProperties(&prop, dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (prop.major != 10) return LAMP_ERR_UNSUPPORTED_DEVICE;
  // table index = shift byte (ue5m3, bias 15): value 2^(E-15)(1 + M/8), E = 0: 2^-14 M/8
  uint32_t lut[256];
  for (int p = 0; p < 256; ++p) {
    const int E = p >> 3, M = p & 7;
    const double s = E ? ldexp(1.0 + M / 8.0, E - 15) : ldexp(M / 8.0, -14);
    lut[p] = exp8_entry(s);
  }
  e = cudaMemcpyToSymbol(c_lut8, lut, sizeof(lut));
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaFuncSetAttribute(lamp_fwd_simt<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)simt_smem_bytes<128>());
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaFuncSetAttribute(lamp_fwd_simt<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)simt_smem_bytes<128>());
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 64) g_init.ready[dev] = true;
  return LAMP_OK;
}

static bool strides_ok(const int64_t* s, int D) {
  return s[0] >= 0 && s[1] >= 0 && s[2] >= D && s[0] % 8 == 0 && s[1] % 8 == 0 && s[2] % 8 == 0;
}

}  // namespace lamp

using namespace lamp;

extern "C" {

int lamp_attn_default_params(lamp_attn_params* p) {
  if (!p) return LAMP_ERR_INVALID_ARG;
  memset(p, 0, sizeof(*p));
  p->causal = 1;
  p->threshold = 0.5f;
  p->delta = 0.00390625f;
  return LAMP_OK;
}

int lamp_attn_contiguous_strides(lamp_attn_params* p) {
  if (!p || p->seqlen <= 0 || p->head_dim <= 0 || p->heads_q <= 0 || p->heads_kv <= 0)
    return LAMP_ERR_INVALID_ARG;
  const int64_t row = p->head_dim, head = row * p->seqlen;
  p->q_strides[0] = head * p->heads_q; p->q_strides[1] = head; p->q_strides[2] = row;
  p->o_strides[0] = head * p->heads_q; p->o_strides[1] = head; p->o_strides[2] = row;
  p->k_strides[0] = head * p->heads_kv; p->k_strides[1] = head; p->k_strides[2] = row;
  p->v_strides[0] = head * p->heads_kv; p->v_strides[1] = head; p->v_strides[2] = row;
  return LAMP_OK;
}

size_t lamp_attn_workspace_bytes(const lamp_attn_params* p) {
  (void)p;
  return 0;
}

static int check_params(const void* q, const void* k, const void* v, void* out,
                        const lamp_attn_params* p) {
  if (!q || !k || !v || !out || !p) return LAMP_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->heads_q <= 0 || p->heads_kv <= 0 || p->seqlen <= 0)
    return LAMP_ERR_INVALID_ARG;
  if (p->heads_q % p->heads_kv) return LAMP_ERR_INVALID_ARG;
  if (!(p->threshold >= 0.0f) || !(p->delta >= 0.0f) || !isfinite(p->scale)) return LAMP_ERR_INVALID_ARG;
  if (p->window < 0 || (p->window > 0 && !p->causal)) return LAMP_ERR_INVALID_ARG;
  if (p->flags & ~(LAMP_FORCE_16BIT | LAMP_FORCE_8BIT | LAMP_NO_STAGE1 | LAMP_OUT_FP32))
    return LAMP_ERR_INVALID_ARG;
  if ((p->flags & LAMP_FORCE_16BIT) && (p->flags & (LAMP_FORCE_8BIT | LAMP_NO_STAGE1)))
    return LAMP_ERR_INVALID_ARG;
  if ((p->dbg_y8 || p->dbg_e8) &&
      (p->dbg_batch < 0 || p->dbg_batch >= p->batch || p->dbg_head < 0 || p->dbg_head >= p->heads_q))
    return LAMP_ERR_INVALID_ARG;
  if (p->head_dim != 128) return LAMP_ERR_UNSUPPORTED_SHAPE;
  if (p->seqlen % kBM) return LAMP_ERR_UNSUPPORTED_SHAPE;
  if (p->batch > 65535 || p->heads_q > 65535) return LAMP_ERR_UNSUPPORTED_SHAPE;
  const int D = p->head_dim;
  if (!strides_ok(p->q_strides, D) || !strides_ok(p->k_strides, D) ||
      !strides_ok(p->v_strides, D) || !strides_ok(p->o_strides, D))
    return LAMP_ERR_UNSUPPORTED_SHAPE;
  if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) return LAMP_ERR_UNSUPPORTED_SHAPE;
  return LAMP_OK;
}

int lamp_attn_fwd(const void* q, const void* k, const void* v, void* out, float* lse,
                  uint8_t* flag_mask, const lamp_attn_params* p, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
  (void)workspace; (void)workspace_bytes;
  int rc = check_params(q, k, v, out, p);
  if (rc) return rc;
  int dev;
  rc = ensure_device(&dev);
  if (rc) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;

  KernelParams P;
  P.q = (const __nv_bfloat16*)q; P.k = (const __nv_bfloat16*)k; P.v = (const __nv_bfloat16*)v;
  P.out = out; P.lse = lse; P.flag_mask = flag_mask;
  for (int i = 0; i < 3; ++i) {
    P.qs[i] = p->q_strides[i]; P.ks[i] = p->k_strides[i];
    P.vs[i] = p->v_strides[i]; P.os[i] = p->o_strides[i];
  }
  P.batch = p->batch; P.heads_q = p->heads_q; P.heads_kv = p->heads_kv; P.seqlen = p->seqlen;
  P.causal = p->causal ? 1 : 0; P.window = p->window;
  P.scale = p->scale; P.tau = p->threshold; P.delta = p->delta; P.flags = p->flags;
  P.dbg_batch = p->dbg_batch; P.dbg_head = p->dbg_head;
  P.dbg_y8 = p->dbg_y8; P.dbg_e8 = p->dbg_e8;
  P.dbg_checksums = (unsigned long long*)p->dbg_checksums;

  void* stats_ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&stats_ptr, g_stats);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaMemsetAsync(stats_ptr, 0, sizeof(DeviceStats), stream);
  if (e != cudaSuccess) return cuda_fail(e);

  const size_t ngt = (size_t)p->batch * p->heads_q * (p->seqlen / kBQ) * (p->seqlen / kTK);
  if (flag_mask) {
    e = cudaMemsetAsync(flag_mask, 0, ngt, stream);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (p->dbg_checksums) {
    e = cudaMemsetAsync(p->dbg_checksums, 0, ngt * 16, stream);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const bool dump = p->dbg_y8 || p->dbg_e8 || p->dbg_checksums;
  dim3 grid(p->seqlen / kBM, p->heads_q, p->batch), block(128);
  const size_t smem = simt_smem_bytes<128>();
  if (dump) lamp_fwd_simt<128, true><<<grid, block, smem, stream>>>(P);
  else lamp_fwd_simt<128, false><<<grid, block, smem, stream>>>(P);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  return LAMP_OK;
}

int lamp_attn_get_stats(lamp_attn_stats* host_out, void* cuda_stream) {
  if (!host_out) return LAMP_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaStreamSynchronize(stream);
  if (e != cudaSuccess) return cuda_fail(e);
  DeviceStats ds;
  e = cudaMemcpyFromSymbol(&ds, g_stats, sizeof(ds));
  if (e != cudaSuccess) return cuda_fail(e);
  memset(host_out, 0, sizeof(*host_out));
  host_out->subblocks_active = ds.v[0];
  host_out->stage1_flagged = ds.v[1];
  host_out->stage2_flagged = ds.v[2];
  for (int i = 0; i < 5; ++i) host_out->hist_flagged_per_tile[i] = ds.v[3 + i];
  host_out->sat_e4m3 = ds.v[8];
  host_out->sat_e4m11 = ds.v[9];
  host_out->exp16_gt1 = ds.v[10];
  host_out->big_rowsum = ds.v[11];
  host_out->device_status = ds.status;
  return ds.status ? LAMP_ERR_DEVICE_TIMEOUT : LAMP_OK;
}

int lamp_attn_last_cuda_error(void) { return t_last_cuda; }

const char* lamp_attn_strerror(int code) {
  switch (code) {
    case LAMP_OK: return "ok";
    case LAMP_ERR_INVALID_ARG: return "invalid argument";
    case LAMP_ERR_UNSUPPORTED_SHAPE: return "unsupported shape, stride or alignment";
    case LAMP_ERR_CUDA: return "CUDA runtime error (see lamp_attn_last_cuda_error)";
    case LAMP_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case LAMP_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.x";
    default: return "unknown error";
  }
}

}  // extern "C"
