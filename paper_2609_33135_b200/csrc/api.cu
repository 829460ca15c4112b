// Host-only exports of the C ABI: sizes, layout index maps, diagnostics.
#include "common.cuh"

using namespace mpfa;

extern "C" size_t mpfa_fp4_codes_bytes(int B, int H, int N) {
  if (B <= 0 || H <= 0 || N <= 0) return 0;
  return (size_t)B * H * pad128(N) * 64;
}

extern "C" size_t mpfa_fp4_sf_bytes(int B, int H, int N) {
  if (B <= 0 || H <= 0 || N <= 0) return 0;
  return (size_t)B * H * (pad128(N) / TILE) * 1024;
}

extern "C" size_t mpfa_delta_s_bytes(int B, int H_q, int N_kv) {
  if (B <= 0 || H_q <= 0 || N_kv <= 0) return 0;
  return (size_t)B * H_q * pad128(N_kv) * 2;
}

extern "C" size_t mpfa_v_fp8_bytes(int B, int H_kv, int N_kv) {
  if (B <= 0 || H_kv <= 0 || N_kv <= 0) return 0;
  return (size_t)B * H_kv * pad128(N_kv) * HEAD_DIM;
}

extern "C" size_t mpfa_sf_offset(int H, int N, int b, int h, int token, int block) {
  const int tiles = pad128(N) / TILE;
  const int r = token % TILE;
  return (((size_t)b * H + h) * tiles + token / TILE) * 1024 + (size_t)(block / 4) * 512 + (r % 32) * 16 +
         (r / 32) * 4 + (block % 4);
}

extern "C" size_t mpfa_paged_k_offset(int token, int block, int byte_in_block) {
  const int r = token % 8;
  return (size_t)(token / 8) * 512 + r * 64 + (((block / 2) ^ (r / 2)) * 16) + (block % 2) * 8 + byte_in_block;
}

extern "C" size_t mpfa_paged_v_offset(int token, int channel) {
  const int r = token % 8;
  return (size_t)(token / 8) * 1024 + r * 128 + (((channel / 16) ^ r) * 16) + channel % 16;
}

extern "C" const char *mpfa_status_string(mpfa_status s) {
  switch (s) {
    case MPFA_OK: return "ok";
    case MPFA_ERR_INVALID_ARG: return "invalid argument";
    case MPFA_ERR_UNSUPPORTED: return "unsupported shape or option";
    case MPFA_ERR_ALIGNMENT: return "misaligned buffer";
    case MPFA_ERR_WORKSPACE: return "workspace too small";
    case MPFA_ERR_ARCH: return "device is not compute capability 10.x";
    case MPFA_ERR_CUDA: return "CUDA call failed";
    case MPFA_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

extern "C" int mpfa_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" int mpfa_version(void) { return 100; }
