// Offline weight preparation: per-out-channel symmetric round-to-nearest codes, permuted and
// padded to the layer's group-contiguous code layout, int4 packed two per byte, plus the
// per-group column sums the de-quantizer needs.  Runs on the host; not a timed path.
#pragma once

#include "groups.cuh"

struct dgq_weight {
  int N = 0, K = 0, C = 0, G = 0, w_bits = 8, is_conv = 0;
  int N_pad = 0;                 // N rounded up to a multiple of 256 (rows beyond N are zero)
  int Kt = 0;                    // length of the GEMM reduction in padded positions (multiple of 32)
  std::vector<int32_t> seg_end;  // [G] end of every group's segment, in 32-position atoms
  std::vector<int8_t> wq;        // host codes, original order [N][K]
  std::vector<float> sw;         // host scales [N]
  int8_t* d_w = nullptr;         // 8-bit: [N_pad][Kt] s8; 4-bit: [N_pad][Kt/2] packed
  float* d_sw = nullptr;         // [N_pad]; 4-bit: sw / 16 (the unpacked codes carry a factor 16)
  float* d_wsum = nullptr;       // [G][N_pad] column sums per group as fp32 (exact); 4-bit: x 16
  float* d_wres = nullptr;       // [G][N_pad] part of wsum the padding positions could not absorb
  uint32_t res_mask = 0;         // bit g set: group g has a non-zero entry in d_wres
};

namespace dgq {

// 4-bit storage: every 8 consecutive positions k0..k0+7 share one 32-bit word whose byte i holds
// code k0+i in its low nibble and code k0+4+i in its high nibble.  In the kernel
// (word << 4) & 0xF0F0F0F0 and word & 0xF0F0F0F0 are then bytes k0..k0+3 and k0+4..k0+7, each
// equal to 16 x the signed code, with no per-byte sign extension.
static void pack_int4_words(const int8_t* row, int Kt, uint8_t* out) {
  for (int k0 = 0; k0 < Kt; k0 += 8)
    for (int i = 0; i < 4; ++i)
      out[k0 / 2 + i] = (uint8_t)((row[k0 + i] & 0x0F) | ((row[k0 + 4 + i] & 0x0F) << 4));
}

static dgq_status weight_build(const dgq_groups* g, const int8_t* wq, const float* sw, int N, int K, int w_bits,
                               const dgq_conv_desc* conv, dgq_weight** out) {
  if (!g || !wq || !sw || !out || N <= 0) return DGQ_ERR_INVALID_ARG;
  if (w_bits != 8 && w_bits != 4) return DGQ_ERR_INVALID_ARG;
  const int taps = conv ? 9 : 1;
  if (conv && (conv->c != g->C || conv->n <= 0 || conv->h <= 0 || conv->w <= 0)) return DGQ_ERR_INVALID_ARG;
  if (K != taps * g->C) return DGQ_ERR_INVALID_ARG;
  if ((N % 8) != 0) return DGQ_ERR_UNSUPPORTED;
  const int qmax = (1 << (w_bits - 1)) - 1;
  for (size_t i = 0; i < (size_t)N * K; ++i)
    if (wq[i] < -qmax || wq[i] > qmax) return DGQ_ERR_INVALID_ARG;
  dgq_weight* w = new dgq_weight();
  w->N = N;
  w->K = K;
  w->C = g->C;
  w->G = g->G;
  w->w_bits = w_bits;
  w->is_conv = conv ? 1 : 0;
  w->N_pad = (N + 255) / 256 * 256;
  w->Kt = taps * g->K_pad;
  // accumulator bound: |code| <= 255, |weight| <= 127 (4-bit: 7 * 16)
  if ((int64_t)w->Kt * 255 * 127 >= ((int64_t)1 << 31)) {
    delete w;
    return DGQ_ERR_UNSUPPORTED;
  }
  w->wq.assign(wq, wq + (size_t)N * K);
  w->sw.assign(sw, sw + N);
  w->seg_end.resize(g->G);
  // GEMM reduction order: group-major; inside a group tap-major (conv), then the group's padded positions
  std::vector<int8_t> Wp((size_t)w->N_pad * w->Kt, 0);
  std::vector<float> wsum((size_t)g->G * w->N_pad, 0.f), wres((size_t)g->G * w->N_pad, 0.f);
  const float unit = (w_bits == 4) ? 16.f : 1.f;
  int pos = 0;
  for (int k = 0; k < g->G; ++k) {
    const int p0 = g->group_off[k], p1 = g->group_off[k + 1];
    for (int t = 0; t < taps; ++t)
      for (int p = p0; p < p1; ++p, ++pos) {
        const int c = g->perm[p];
        if (c < 0) continue;
        for (int o = 0; o < N; ++o) Wp[(size_t)o * w->Kt + pos] = wq[(size_t)o * K + t * g->C + c];
      }
    w->seg_end[k] = pos / DGQ_K_ATOM;
    const int seg0 = pos - taps * (p1 - p0);  // first reduction position of this group
    for (int o = 0; o < N; ++o) {
      int64_t sum = 0;
      for (int c = 0; c < g->C; ++c)
        if (g->col_group[c] == k)
          for (int t = 0; t < taps; ++t) sum += wq[(size_t)o * K + t * g->C + c];
      wsum[(size_t)k * w->N_pad + o] = (float)sum * unit;
      // Linear layers: spread -sum over the group's padding positions (whose activation code is the
      // zero-point Z), so that acc + Z * (-sum) = acc - Z * wsum comes out of the integer product.
      // What does not fit in the available positions stays in `wres` for the epilogue.
      int64_t rem = conv ? 0 : -sum;
      if (!conv)
        for (int p = p0; p < p1 && rem != 0; ++p)
          if (g->perm[p] < 0) {
            const int64_t v = std::max<int64_t>(-qmax, std::min<int64_t>(qmax, rem));
            Wp[(size_t)o * w->Kt + seg0 + (p - p0)] = (int8_t)v;
            rem -= v;
          }
      const int64_t res = conv ? sum : -rem;  // conv uses zero-centred codes: no zero-point term at all
      wres[(size_t)k * w->N_pad + o] = (float)res * unit;
      if (res != 0 && !conv) w->res_mask |= 1u << k;
    }
  }
  std::vector<float> swp(w->N_pad, 0.f);
  for (int o = 0; o < N; ++o) swp[o] = sw[o] / unit;
  dgq_status st = DGQ_OK;
  auto up = [&](void** d, const void* h, size_t bytes) {
    if (st != DGQ_OK) return;
    if (cudaMalloc(d, bytes) != cudaSuccess || cudaMemcpy(*d, h, bytes, cudaMemcpyHostToDevice) != cudaSuccess)
      st = DGQ_ERR_CUDA;
  };
  if (w_bits == 8) {
    up((void**)&w->d_w, Wp.data(), Wp.size());
  } else {
    std::vector<uint8_t> packed((size_t)w->N_pad * w->Kt / 2);
    for (int o = 0; o < w->N_pad; ++o)
      pack_int4_words(&Wp[(size_t)o * w->Kt], w->Kt, &packed[(size_t)o * w->Kt / 2]);
    up((void**)&w->d_w, packed.data(), packed.size());
  }
  up((void**)&w->d_sw, swp.data(), swp.size() * sizeof(float));
  up((void**)&w->d_wsum, wsum.data(), wsum.size() * sizeof(float));
  up((void**)&w->d_wres, wres.data(), wres.size() * sizeof(float));
  if (st != DGQ_OK) {
    cudaFree(w->d_w);
    cudaFree(w->d_sw);
    cudaFree(w->d_wsum);
    cudaFree(w->d_wres);
    delete w;
    return st;
  }
  *out = w;
  return DGQ_OK;
}

}  // namespace dgq

extern "C" dgq_status dgq_weight_from_codes(const dgq_groups* g, const int8_t* wq, const float* sw, int N, int K,
                                            int w_bits, const dgq_conv_desc* conv, dgq_weight** out) {
  return dgq::weight_build(g, wq, sw, N, K, w_bits, conv, out);
}

extern "C" dgq_status dgq_weight_prepare(const dgq_groups* g, const void* W, int N, int K, int w_bits,
                                         const dgq_conv_desc* conv, dgq_weight** out, void* stream) {
  if (!g || !W || !out || N <= 0 || K <= 0) return DGQ_ERR_INVALID_ARG;
  if (w_bits != 8 && w_bits != 4) return DGQ_ERR_INVALID_ARG;
  std::vector<__half> h((size_t)N * K);
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return DGQ_ERR_CUDA;
  if (cudaMemcpy(h.data(), W, h.size() * sizeof(__half), cudaMemcpyDeviceToHost) != cudaSuccess)
    return DGQ_ERR_CUDA;
  // fp32 sequence: sw = absmax / qmax, inv = 1 / sw, code = clamp(rint(w * inv), -qmax, qmax)
  const float qmax = (float)((1 << (w_bits - 1)) - 1);
  std::vector<int8_t> wq((size_t)N * K);
  std::vector<float> sw(N);
  for (int o = 0; o < N; ++o) {
    float amax = 0.f;
    for (int k = 0; k < K; ++k) amax = std::max(amax, std::fabs(__half2float(h[(size_t)o * K + k])));
    volatile float s = amax > 0.f ? amax / qmax : 1.0f;
    volatile float inv = 1.0f / s;
    sw[o] = s;
    for (int k = 0; k < K; ++k) {
      volatile float t = __half2float(h[(size_t)o * K + k]) * inv;
      float r = __builtin_rintf(t);
      r = std::min(std::max(r, -qmax), qmax);
      wq[(size_t)o * K + k] = (int8_t)r;
    }
  }
  return dgq::weight_build(g, wq.data(), sw.data(), N, K, w_bits, conv, out);
}

extern "C" dgq_status dgq_weight_destroy(dgq_weight* w) {
  if (!w) return DGQ_OK;
  cudaFree(w->d_w);
  cudaFree(w->d_sw);
  cudaFree(w->d_wsum);
  cudaFree(w->d_wres);
  delete w;
  return DGQ_OK;
}

extern "C" dgq_status dgq_weight_export(const dgq_weight* w, int8_t* wq, float* sw) {
  if (!w) return DGQ_ERR_INVALID_ARG;
  if (wq) std::copy(w->wq.begin(), w->wq.end(), wq);
  if (sw) std::copy(w->sw.begin(), w->sw.end(), sw);
  return DGQ_OK;
}
