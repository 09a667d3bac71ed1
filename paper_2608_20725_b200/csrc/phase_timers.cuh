// Phase timers of the fp16 kernels: a measuring aid that exists only in builds made with
// -DIM2WIN_F16_TIMERS (never the library that ships).  In such a build each role of a kernel adds the
// clock64 cycles it spends per phase into the 64-bit words 4.. of the status block (CTA 0 only);
// in every other build the three macros expand to nothing.
#pragma once

#ifdef IM2WIN_F16_TIMERS
// Debug build only: per-thread cycle counters, flushed once into the 64-bit words 4.. of the status block.
#define TIMER_DECL long long t_prev = clock64(), t_now, t_acc[20] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define TIMER_LAP(slot)                 \
  do {                                  \
    t_now = clock64();                  \
    t_acc[slot] += t_now - t_prev;      \
    t_prev = t_now;                     \
  } while (0)
#define TIMER_FLUSH()                                                                                              \
  do {                                                                                                             \
    for (int ti = 0; ti < 20; ++ti)                                                                                \
      if (t_acc[ti]) atomicAdd(reinterpret_cast<unsigned long long*>(q.status) + 4 + ti, (unsigned long long)t_acc[ti]); \
  } while (0)
#else
#define TIMER_DECL
#define TIMER_LAP(slot)
#define TIMER_FLUSH()
#endif
