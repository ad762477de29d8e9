// Cycle accounting for profiling builds of the GEMM kernel (-DQG_PROFILE): every role adds the cycles it spends
// in each of its waits to a per-CTA counter block.  In the product build all of these expand to nothing.
#pragma once

#if defined(QG_PROFILE)
#define QG_T0() long long qg_t0_ = clock64()
#define QG_ACC(slot) do { if (p.stats) { long long now_ = clock64(); qg_stat_[slot] += now_ - qg_t0_; qg_t0_ = now_; } } while (0)
#define QG_DECL() long long qg_stat_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define QG_FLUSH() do { if (p.stats) for (int i_ = 0; i_ < 12; ++i_) if (qg_stat_[i_]) atomicAdd(reinterpret_cast<unsigned long long*>(p.stats) + blockIdx.x * 12 + i_, static_cast<unsigned long long>(qg_stat_[i_])); } while (0)
#else
#define QG_T0() do {} while (0)
#define QG_ACC(slot) do {} while (0)
#define QG_DECL() do {} while (0)
#define QG_FLUSH() do {} while (0)
#endif
