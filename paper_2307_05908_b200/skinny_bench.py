"""Times the two skinny-product kernels side by side on one GPU: the FMA kernel of the decode path
(ppd_op_gemv) and the experimental tensor-core form (ppd_op_gemv_tc), for M = 1, 3, 5, 8 rows on the
matrix shapes of the 7B-shaped model.  Each call streams a different weight matrix (12 of them, far
more than L2 holds), CUDA events on the launching stream, best of 5.

    python -m paper_2307_05908_b200.skinny_bench

The tensor-core entry point runs two kernels per call (RMSNorm + split of the activation rows, then
the product); the product kernel alone is what a launch list shows (profiles/)."""
from __future__ import annotations

import torch

import paper_2307_05908_b200 as ppd

DEV = "cuda:0"
SHAPES = ((22016, 4096, "gate/up"), (12288, 4096, "qkv"), (4096, 11008, "down"))


def run(N, K, name, n_mats=12, reps=5):
    nbytes = ppd.packed_bytes(N, K)
    tcb = ppd.load().ppd_op_tc_packed_bytes(N, K)
    mats = [torch.randint(0, 2 ** 14, (max(nbytes, tcb) // 2,), dtype=torch.int16, device=DEV) for _ in range(n_mats)]
    Kp = (K + 255) // 256 * 256
    for M in (1, 3, 5, 8):
        x = torch.randn(M, Kp, device=DEV)
        out = torch.zeros(M, N, device=DEV)
        scratch = torch.zeros(ppd.op_gemv_tc_scratch_bytes(K), dtype=torch.uint8, device=DEV)
        res = {}
        for kind in ("fma", "tc"):
            def one(w):
                if kind == "fma":
                    ppd.op_gemv(w, N, K, x, None, 1e-5, 0, None, out)
                else:
                    ppd.op_gemv_tc(w, N, K, x, None, 1e-5, out, scratch)
            for w in mats:
                one(w)
            torch.cuda.synchronize()
            best = 1e9
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for w in mats:
                    one(w)
                e1.record()
                torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1) / n_mats)
            res[kind] = best
        print(f"{name} N={N} K={K} M={M}: FMA kernel {res['fma'] * 1e3:.1f} us ({nbytes / res['fma'] / 1e6:.0f} GB/s), "
              f"tensor-core entry point (2 kernels) {res['tc'] * 1e3:.1f} us", flush=True)


def main():
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    for N, K, name in SHAPES:
        run(N, K, name)


if __name__ == "__main__":
    main()
