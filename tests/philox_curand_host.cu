// Test helper: prints cuRAND's own Philox4x32-10 block function evaluated on the host, so the
// oracle's generator can be checked against the vendor header without a GPU.
// usage: philox_curand_host < lines of "c0 c1 c2 c3 k0 k1" (hex)  ->  lines of "o0 o1 o2 o3" (hex)
#define QUALIFIERS static inline __host__ __device__
#include <cstdio>
#include <cuda_runtime.h>
#include <curand_philox4x32_x.h>

int main() {
  unsigned c0, c1, c2, c3, k0, k1;
  while (std::scanf("%x %x %x %x %x %x", &c0, &c1, &c2, &c3, &k0, &k1) == 6) {
    uint4 c = make_uint4(c0, c1, c2, c3);
    uint2 k = make_uint2(k0, k1);
    uint4 o = curand_Philox4x32_10(c, k);
    std::printf("%08x %08x %08x %08x\n", o.x, o.y, o.z, o.w);
  }
  return 0;
}
