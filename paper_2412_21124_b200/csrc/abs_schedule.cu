// Host-side batch-size schedule (Algorithm 1: the If branch's rounding and the loop counters;
// Sec. 5: maximum global batch size and test interval; Tables 5-7: maximum micro batch size).
// Pure integer arithmetic; nothing here touches the device.
#include "../../include/abs_normtest.h"

namespace {

constexpr int64_t kLimit = int64_t{1} << 60;

int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// a*b, or -1 when it would pass 2^60
int64_t mul_checked(int64_t a, int64_t b) {
  if (a < 1 || b < 1 || a > kLimit / b) return -1;
  return a * b;
}

}  // namespace

extern "C" {

int abs_schedule_init(abs_schedule* s, int64_t J, int64_t M, int64_t micro0, int64_t b_max,
                      int64_t max_micro, int64_t interval) {
  if (!s) return ABS_ERR_NULL;
  if (J < 1 || M < 1 || micro0 < 1 || b_max < 1 || max_micro < 0 || interval < 1)
    return ABS_ERR_RANGE;
  if (max_micro > 0 && micro0 > max_micro) return ABS_ERR_RANGE;
  if (b_max > kLimit) return ABS_ERR_RANGE;
  const int64_t jm = mul_checked(J, M);
  const int64_t b0 = jm < 0 ? -1 : mul_checked(jm, micro0);
  if (b0 < 0 || b0 > b_max) return ABS_ERR_RANGE;
  s->J = J;
  s->M = M;
  s->micro = micro0;
  s->b = b0;
  s->b_max = b_max;
  s->max_micro = max_micro;
  s->interval = interval;
  s->step = 1;
  s->samples = 0;
  return ABS_OK;
}

int abs_schedule_test_due(const abs_schedule* s) {
  if (!s) return -1;
  return (s->b < s->b_max && s->step % s->interval == 0) ? 1 : 0;
}

int abs_schedule_advance(abs_schedule* s, int64_t b_test) {
  if (!s) return ABS_ERR_NULL;
  if (b_test < 1) return ABS_ERR_RANGE;
  const int64_t used = s->b;
  const int64_t target = b_test < s->b_max ? b_test : s->b_max;
  if (target > s->b) {
    // J*M <= b <= b_max <= 2^60, so every product below stays under 2^62
    int64_t M = s->M;
    int64_t micro = ceil_div(target, s->J * M);
    if (s->max_micro > 0 && micro > s->max_micro) {
      M = ceil_div(target, s->J * s->max_micro);
      micro = ceil_div(target, s->J * M);
    }
    int64_t b = s->J * M * micro;
    if (b > s->b_max) {
      micro = s->b_max / (s->J * M);
      b = s->J * M * micro;
    }
    if (micro >= 1 && b > s->b) {
      s->M = M;
      s->micro = micro;
      s->b = b;
    }
  }
  s->samples += used;
  s->step += 1;
  return ABS_OK;
}

}  // extern "C"
