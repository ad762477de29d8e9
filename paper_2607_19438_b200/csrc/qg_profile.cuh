// Cycle accounting for profiling builds of the GEMM kernel (-DQG_PROFILE): every role adds the cycles it spends
// in each of its waits to a per-CTA counter block.  In the product build all of these expand to nothing.
#pragma once

#if defined(QG_PROFILE)
#define QG_T0() long long qg_t0_ = clock64()
#define QG_ACC(slot) do { if (p.stats) { long long now_ = clock64(); qg_stat_[slot] += now_ - qg_t0_; qg_t0_ = now_; } } while (0)
#define QG_DECL() long long qg_stat_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define QG_FLUSH() do { if (p.stats) for (int i_ = 0; i_ < 12; ++i_) if (qg_stat_[i_]) atomicAdd(reinterpret_cast<unsigned long long*>(p.stats) + blockIdx.x * 12 + i_, static_cast<unsigned long long>(qg_stat_[i_])); } while (0)
// Milestones of the first CTA (one clock64 stamp per index, written by whichever thread reaches the call site first
// in program order of its role), after the 148 x 12 wait counters.
#define QG_MARK(idx) do { if (p.stats && blockIdx.x == 0 && (threadIdx.x & 31) == 0) p.stats[148 * 12 + (idx)] = clock64(); } while (0)
// Wall-clock (globaltimer, ns) entry and exit stamps of every CTA, after the milestones.
#define QG_SPAN(which) do { if (p.stats && threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); p.stats[148 * 12 + 16 + 2 * blockIdx.x + (which)] = static_cast<long long>(t_); } } while (0)
#else
#define QG_SPAN(which) do {} while (0)
#define QG_MARK(idx) do {} while (0)
#define QG_T0() do {} while (0)
#define QG_ACC(slot) do {} while (0)
#define QG_DECL() do {} while (0)
#define QG_FLUSH() do {} while (0)
#endif
