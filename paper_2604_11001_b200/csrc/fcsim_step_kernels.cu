// The step kernels, one policy at a time: the build compiles this file once per policy
// (-DFCSIM_KERNEL_POLICY=0 .. 6) into an object of its own, so that every policy's kernels are optimised as a
// separate module, always the same way, and the objects build side by side on the host's cores.  Each object
// exports one function that hands the host the kernel for a register allocation and a variant.  Compiled without
// the macro, the file holds all seven policies (a plain two-file build: slower to compile, same kernels).
#include "fcsim_device.cuh"

namespace fcsim_dev {

namespace {

// The step kernel of policy kPol compiled for a register allocation that lets 8, 7, 6 or 5 CTAs reside on an SM,
// for what is recorded per slot (0 nothing, 1 trace only, 2 decided at run time; Algorithm 1 and the MC benchmark
// exist in the run-time form only), for the whole-prompt first-come-first-served policies with or without the
// activation of several queue heads at once, and for policies 0 .. 3 with or without arrivals drawn at the queue
// head.
template <int kPol, int kCtas>
step_kernel_t step_kernel_for(int rec, bool bulk, bool lazy) {
    constexpr bool kFifo = kPol <= 1 || kPol == 3 || kPol == 6;
    constexpr int kP = kPol >= 4 ? 0 : kPol;  // keeps the specialised forms of policies 4 .. 6 uninstantiated
    if constexpr (kPol <= 3) {
        if (lazy && !bulk) {  // lazily drawn arrivals: without the several-heads step
            if (rec == 2) return fcsim_step_kernel<kP, kCtas, 2, false, true>;
            if (rec == 1) return fcsim_step_kernel<kP, kCtas, 1, false, true>;
            return fcsim_step_kernel<kP, kCtas, 0, false, true>;
        }
    }
    if constexpr (kFifo) {
        if (bulk) {
            if constexpr (kPol >= 4) {
                return fcsim_step_kernel<kPol, kCtas, 2, true, false>;
            } else {
                if (rec == 2) return fcsim_step_kernel<kP, kCtas, 2, true, false>;
                if (rec == 1) return fcsim_step_kernel<kP, kCtas, 1, true, false>;
                return fcsim_step_kernel<kP, kCtas, 0, true, false>;
            }
        }
    }
    if constexpr (kPol >= 4) {
        return fcsim_step_kernel<kPol, kCtas, 2, false, false>;
    } else {
        if (rec == 2) return fcsim_step_kernel<kP, kCtas, 2, false, false>;
        if (rec == 1) return fcsim_step_kernel<kP, kCtas, 1, false, false>;
        return fcsim_step_kernel<kP, kCtas, 0, false, false>;
    }
}

template <int kPol>
step_kernel_t step_kernel_of_policy(int ctas, int rec, bool bulk, bool lazy) {
    switch (ctas) {
        case 8: return step_kernel_for<kPol, 8>(rec, bulk, lazy);
        case 5: return step_kernel_for<kPol, 5>(rec, bulk, lazy);
        case 6: return step_kernel_for<kPol, 6>(rec, bulk, lazy);
        default: return step_kernel_for<kPol, 7>(rec, bulk, lazy);
    }
}

}  // namespace

#define FCSIM_EXPORT_POLICY2(n)                                                          \
    step_kernel_t step_kernel_of_policy_##n(int ctas, int rec, bool bulk, bool lazy) {  \
        return step_kernel_of_policy<n>(ctas, rec, bulk, lazy);                         \
    }
#define FCSIM_EXPORT_POLICY(n) FCSIM_EXPORT_POLICY2(n)

#ifdef FCSIM_KERNEL_POLICY
FCSIM_EXPORT_POLICY(FCSIM_KERNEL_POLICY)
#else
FCSIM_EXPORT_POLICY(0)
FCSIM_EXPORT_POLICY(1)
FCSIM_EXPORT_POLICY(2)
FCSIM_EXPORT_POLICY(3)
FCSIM_EXPORT_POLICY(4)
FCSIM_EXPORT_POLICY(5)
FCSIM_EXPORT_POLICY(6)
#endif

}  // namespace fcsim_dev
