// Host build of the kernels' scalar math (ersd_math.cuh) so that the error
// bounds the kernels rely on can be checked without a GPU.  Not part of libersd.so.
#include "ersd_math.cuh"

extern "C" {
void ersd_host_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  ersd::philox4x32_10(ctr[0], ctr[1], ctr[2], ctr[3], key[0], key[1], out);
}
uint32_t ersd_host_token_word(uint64_t seed, uint32_t seq, uint32_t pos, uint32_t i) {
  return ersd::token_word(seed, seq, pos, i);
}
void ersd_host_philox_row(uint64_t seed, uint32_t seq, uint32_t pos, uint32_t c0, uint32_t* out) {
  ersd::PhiloxRow pr;
  pr.init(seed, seq, pos);
  pr.words(c0, out);
}
double ersd_host_exact_ln_e(uint32_t x) { return ersd::exact_ln_e(x); }
double ersd_host_exact_key(uint32_t x, float z, float T) { return ersd::exact_key(x, z, T); }
float ersd_host_screen_lg2_e(uint32_t x) { return ersd::screen_lg2_e(x); }
float ersd_host_screen_slack(float tau) { return ersd::screen_slack(tau); }
float ersd_host_screen_core(void) { return ersd::kScreenCore; }
// screening key (log2 units) exactly as the kernel forms it
float ersd_host_screen_key(uint32_t x, float z, float T) {
  const float c2 = (float)(1.4426950408889634 / (double)T);
  return fmaf(-z, c2, ersd::screen_lg2_e(x));
}
void ersd_host_screen_lg2_e_many(const uint32_t* x, int n, float* out) {
  for (int i = 0; i < n; ++i) out[i] = ersd::screen_lg2_e(x[i]);
}
}
