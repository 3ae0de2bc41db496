// Shared-memory barrier helpers used by every kernel of the library: the 32-bit shared address
// of a pointer, one non-blocking parity test, and the bounded wait (every wait in this library
// gives up after about a second of SM clock instead of spinning for ever).
#pragma once
#include <stdint.h>

namespace delta {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
constexpr long long kWaitBudgetClocks = 2000000000ll;
// Bounded wait; false if it ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitBudgetClocks) return false;
  }
  return true;
}
// Bounded wait with a CTA-wide abort flag: a wait that runs out raises the flag, and once the
// flag is up every wait returns at once, so the CTA's protocol still runs to its end.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag) return;
    if (clock64() - t0 > kWaitBudgetClocks) { *abort_flag = 1; return; }
  }
}

// The same bounded wait as a tight poll (mbarrier.test_wait returns at once where try_wait may
// suspend the thread for a while): for the single threads that issue tensor-core work, whose
// reaction time is on the critical path of every tile.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mbar_poll(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test_wait(bar, parity)) return;
  const long long t0 = clock64();
  unsigned spins = 0;
  while (!mbar_test_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*abort_flag) return;
      if (clock64() - t0 > kWaitBudgetClocks) { *abort_flag = 1; return; }
    }
  }
}

}  // namespace delta
