// Test-only helper: prints Philox4x32-10 blocks from two independent
// third-party host engines that ship in this image's headers, so that the
// oracle's from-specification implementation can be compared with them.
//   philox_ref torch <seed> <subsequence> <offset>   -> 4 words (at::philox_engine)
//   philox_ref std   <seed32> <c3> <c2> <c1> <c0>    -> 4 words (cuda::std::philox4x32 after set_counter)
#include <cstdio>
#include <cstdlib>
#include <cstring>
#ifdef HAVE_TORCH_PHILOX
#include <ATen/core/PhiloxRNGEngine.h>
#endif
#ifdef HAVE_STD_PHILOX
#include <cuda/std/__random/philox_engine.h>
#endif

int main(int argc, char** argv) {
  if (argc < 2) return 2;
#ifdef HAVE_TORCH_PHILOX
  if (!strcmp(argv[1], "torch") && argc == 5) {
    at::philox_engine e(strtoull(argv[2], 0, 10), strtoull(argv[3], 0, 10), strtoull(argv[4], 0, 10));
    unsigned a = e(), b = e(), c = e(), d = e();
    printf("%u %u %u %u\n", a, b, c, d);
    return 0;
  }
#endif
#ifdef HAVE_STD_PHILOX
  if (!strcmp(argv[1], "std") && argc == 7) {
    cuda::std::philox4x32 e((unsigned)strtoul(argv[2], 0, 10));
    e.set_counter({(unsigned)strtoul(argv[3], 0, 10), (unsigned)strtoul(argv[4], 0, 10),
                   (unsigned)strtoul(argv[5], 0, 10), (unsigned)strtoul(argv[6], 0, 10)});
    unsigned a = e(), b = e(), c = e(), d = e();
    printf("%u %u %u %u\n", a, b, c, d);
    return 0;
  }
#endif
  return 3;
}
