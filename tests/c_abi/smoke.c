/*
 * The C ABI used from plain C, without Python or torch: a cache of two segments is filled with cudaMemcpy,
 * grown by one row with catekv_append, planned and attended over with catekv_decode_attn; the result is
 * compared with attention written out in C (double precision).  Exit code 0 on success.
 *
 *   gcc -std=c11 -I include -I $CUDA/include tests/c_abi/smoke.c -L paper_2608_30295_b200 -lcatekv \
 *       -L $CUDA/lib64 -lcudart -lm -o smoke
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "catekv.h"

#define D CATEKV_HEAD_DIM
#define CHECK(x)                                                        \
  do {                                                                  \
    if (!(x)) {                                                         \
      fprintf(stderr, "smoke.c:%d: check failed: %s\n", __LINE__, #x);  \
      return 1;                                                         \
    }                                                                   \
  } while (0)

static uint16_t to_bf16(float f) { /* round to nearest even */
  uint32_t u;
  memcpy(&u, &f, 4);
  u += 0x7fffu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}
static double from_bf16(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}
static float rnd(uint32_t* s) { /* small deterministic generator, values in [-1, 1) */
  *s = *s * 1664525u + 1013904223u;
  return (float)((*s >> 8) & 0xffff) / 32768.0f - 1.0f;
}

int main(void) {
  enum { B = 1, HKV = 2, G = 2, HQ = HKV * G, NSEG = B * HKV };
  const int32_t len0[NSEG] = {37, 130};
  int32_t seg_off[NSEG], seg_cap[NSEG], seg_len[NSEG] = {37, 130};
  int64_t total_rows = 0;
  CHECK(catekv_cache_layout(B, HKV, len0, 4, seg_off, seg_cap, &total_rows) == CATEKV_OK);
  CHECK(catekv_version() >= 1000);

  /* host data: pools, one appended row per segment, queries */
  const size_t pool_elems = (size_t)total_rows * D;
  uint16_t* hk = calloc(pool_elems, 2);
  uint16_t* hv = calloc(pool_elems, 2);
  uint16_t hkn[NSEG * D], hvn[NSEG * D], hq[HQ * D];
  uint32_t s = 12345u;
  for (int g = 0; g < NSEG; ++g)
    for (int r = 0; r < len0[g]; ++r)
      for (int e = 0; e < D; ++e) {
        hk[((size_t)seg_off[g] + r) * D + e] = to_bf16(rnd(&s));
        hv[((size_t)seg_off[g] + r) * D + e] = to_bf16(rnd(&s));
      }
  for (int i = 0; i < NSEG * D; ++i) hkn[i] = to_bf16(rnd(&s)), hvn[i] = to_bf16(rnd(&s));
  for (int i = 0; i < HQ * D; ++i) hq[i] = to_bf16(3.0f * rnd(&s));

  void *dk, *dv, *dkn, *dvn, *dq, *dout, *dplan, *dws;
  int32_t *doff, *dlen;
  CHECK(cudaMalloc(&dk, pool_elems * 2) == cudaSuccess && cudaMalloc(&dv, pool_elems * 2) == cudaSuccess);
  CHECK(cudaMalloc(&dkn, sizeof hkn) == cudaSuccess && cudaMalloc(&dvn, sizeof hvn) == cudaSuccess);
  CHECK(cudaMalloc(&dq, sizeof hq) == cudaSuccess && cudaMalloc(&dout, HQ * D * sizeof(float)) == cudaSuccess);
  CHECK(cudaMalloc((void**)&doff, sizeof seg_off) == cudaSuccess && cudaMalloc((void**)&dlen, sizeof seg_len) == cudaSuccess);
  CHECK(cudaMemcpy(dk, hk, pool_elems * 2, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(dv, hv, pool_elems * 2, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(dkn, hkn, sizeof hkn, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(dvn, hvn, sizeof hvn, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(dq, hq, sizeof hq, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(doff, seg_off, sizeof seg_off, cudaMemcpyHostToDevice) == cudaSuccess);
  CHECK(cudaMemcpy(dlen, seg_len, sizeof seg_len, cudaMemcpyHostToDevice) == cudaSuccess);

  catekv_cache cache;
  memset(&cache, 0, sizeof cache);
  cache.B = B, cache.Hkv = HKV, cache.d = D, cache.total_rows = total_rows;
  cache.k_pool = dk, cache.v_pool = dv, cache.seg_off_dev = doff, cache.seg_len_dev = dlen;
  cache.seg_off = seg_off, cache.seg_cap = seg_cap, cache.seg_len = seg_len;

  CHECK(catekv_append(&cache, dkn, dvn, NULL) == CATEKV_OK);
  CHECK(seg_len[0] == 38 && seg_len[1] == 131);

  const int num_ctas = 5;
  const size_t plan_bytes = catekv_decode_plan_bytes(B, HKV, num_ctas);
  const size_t ws_bytes = catekv_decode_workspace_bytes(B, HKV, num_ctas);
  void* plan_host = malloc(plan_bytes);
  CHECK(plan_bytes > 0 && ws_bytes > 0 && plan_host);
  CHECK(cudaMalloc(&dplan, plan_bytes) == cudaSuccess && cudaMalloc(&dws, ws_bytes) == cudaSuccess);
  CHECK(catekv_decode_plan(&cache, num_ctas, plan_host, dplan, plan_bytes, NULL) == CATEKV_OK);
  CHECK(catekv_decode_attn(&cache, dq, HQ, 0.0f, dout, CATEKV_OUT_FP32, NULL, plan_host, dplan, plan_bytes, dws, ws_bytes,
                           NULL) == CATEKV_OK);
  /* argument checks come back as codes, nothing is launched */
  CHECK(catekv_decode_attn(&cache, dq, 3, 0.0f, dout, CATEKV_OUT_FP32, NULL, plan_host, dplan, plan_bytes, dws, ws_bytes,
                           NULL) == CATEKV_ERR_INVALID_ARG);
  float out[HQ * D];
  CHECK(cudaDeviceSynchronize() == cudaSuccess);
  CHECK(cudaMemcpy(out, dout, sizeof out, cudaMemcpyDeviceToHost) == cudaSuccess);

  /* attention in plain C over the same rows (the appended row last) */
  double num = 0.0, den = 0.0, worst = 0.0;
  for (int hq_i = 0; hq_i < HQ; ++hq_i) {
    const int g = hq_i / G, n = len0[g] + 1;
    double* logit = malloc(sizeof(double) * n);
    double mx = -INFINITY;
    for (int r = 0; r < n; ++r) {
      const uint16_t* krow = r < len0[g] ? hk + ((size_t)seg_off[g] + r) * D : hkn + g * D;
      double dot = 0.0;
      for (int e = 0; e < D; ++e) dot += from_bf16(hq[hq_i * D + e]) * from_bf16(krow[e]);
      logit[r] = dot / sqrt((double)D);
      if (logit[r] > mx) mx = logit[r];
    }
    double z = 0.0, o[D];
    memset(o, 0, sizeof o);
    for (int r = 0; r < n; ++r) {
      const uint16_t* vrow = r < len0[g] ? hv + ((size_t)seg_off[g] + r) * D : hvn + g * D;
      const double p = exp(logit[r] - mx);
      z += p;
      for (int e = 0; e < D; ++e) o[e] += p * from_bf16(vrow[e]);
    }
    for (int e = 0; e < D; ++e) {
      const double ref = o[e] / z, got = out[hq_i * D + e];
      num += (got - ref) * (got - ref);
      den += ref * ref;
      if (fabs(got - ref) > worst) worst = fabs(got - ref);
    }
    free(logit);
  }
  const double rel = sqrt(num / den);
  printf("c abi smoke: rel-L2 %.3e, max-abs %.3e\n", rel, worst);
  CHECK(rel <= 1e-3 && worst <= 1e-2);
  return 0;
}
