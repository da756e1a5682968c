// The step kernels of ONE policy: this file is compiled once per policy (-DFCSIM_KERNEL_POLICY=0 .. 6) into an
// object of its own, so that every policy's kernels are optimised as a separate module, always the same way, and
// the objects build side by side on the host's cores.  Each object exports one function that hands the host
// the kernel for a register allocation and a variant.
#include "fcsim_device.cuh"

#ifndef FCSIM_KERNEL_POLICY
#error "compile with -DFCSIM_KERNEL_POLICY=<0 .. 6>"
#endif

namespace fcsim_dev {

namespace {

constexpr int kPol = FCSIM_KERNEL_POLICY;

// The step kernel compiled for a register allocation that lets 8, 7, 6 or 5 CTAs reside on an SM, for what is
// recorded per slot (0 nothing, 1 trace only, 2 decided at run time; Algorithm 1 and the MC benchmark exist in
// the run-time form only), for the whole-prompt first-come-first-served policies with or without the activation of
// several queue heads at once, and for policies 0 .. 3 with or without arrivals drawn at the queue head.
template <int kCtas>
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

}  // namespace

#define FCSIM_PASTE2(a, b) a##b
#define FCSIM_PASTE(a, b) FCSIM_PASTE2(a, b)

step_kernel_t FCSIM_PASTE(step_kernel_of_policy_, FCSIM_KERNEL_POLICY)(int ctas, int rec, bool bulk, bool lazy) {
    switch (ctas) {
        case 8: return step_kernel_for<8>(rec, bulk, lazy);
        case 5: return step_kernel_for<5>(rec, bulk, lazy);
        case 6: return step_kernel_for<6>(rec, bulk, lazy);
        default: return step_kernel_for<7>(rec, bulk, lazy);
    }
}

}  // namespace fcsim_dev
