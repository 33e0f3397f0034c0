"""Seeded synthetic layer stacks generated on the device (input generation only: none of the method's
arithmetic lives here; quantization of the generated weights and projections goes through the library).

The numpy generators of ``synth`` feed the parity tests, where the CPU oracle needs the same bits; a whole
LLaMA-1B or 7B stack is too large to make on the host and copy, so the throughput runs and the full-size tests
draw the same model (rank-32 signal with singular values 1/k plus Gaussian noise, Gaussian weights, an
orthonormal projection) with torch on the GPU."""
from __future__ import annotations

def build_stack(workload, device, seed=0, layers=0, moments=32):
    """Device-resident synthetic state of the whole stack: bf16 gradients (rank-32 signal + noise),
    INT8 weights, INT4 projections, zero moments.  Generated with torch on the device (input
    generation, not the path); quantization goes through the library."""
    import torch
    from . import binding as B
    from . import synth
    specs = synth.stack_matrices(workload)
    if layers:
        specs = [s for s in specs if s.layer < layers]
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    items = []
    sig = 1.0 / torch.arange(1, synth.SIGNAL_RANK + 1, device=device, dtype=torch.float32)
    for s in specs:
        k = min(synth.SIGNAL_RANK, s.m, s.n)
        U = torch.linalg.qr(torch.randn(s.m, k, device=device, generator=gen))[0]
        Vt = torch.linalg.qr(torch.randn(s.n, k, device=device, generator=gen))[0]
        g32 = (U * sig[:k]) @ Vt.T + synth.NOISE_STD * torch.randn(s.m, s.n, device=device, generator=gen)
        G = B.empty_matrix(s.m, s.n, torch.bfloat16, device)
        G.copy_(g32)
        del g32
        w32 = B.empty_matrix(s.m, s.n, torch.float32, device)
        w32.copy_(torch.randn(s.m, s.n, device=device, generator=gen) * synth.WEIGHT_STD)
        W = B.quantize_int8(w32)
        del w32
        p32 = B.empty_matrix(s.m, s.r, torch.float32, device)
        p32.copy_(torch.linalg.qr(torch.randn(s.m, s.r, device=device, generator=gen))[0])
        P = B.quantize_int4(p32)
        del p32
        if moments == 8:        # 8-bit block-wise moments: codes and one scale per 32 columns, all zero at the start
            M = B.zeros_matrix(s.r, s.n, torch.int8, device)
            V = B.zeros_matrix(s.r, s.n, torch.uint8, device)
            extra = {"M_scale": torch.zeros((s.r, (s.n + 31) // 32), dtype=torch.float32, device=device),
                     "V_scale": torch.zeros((s.r, (s.n + 31) // 32), dtype=torch.float32, device=device)}
        else:
            M = B.zeros_matrix(s.r, s.n, torch.float32, device)
            V = B.zeros_matrix(s.r, s.n, torch.float32, device)
            extra = {}
        items.append({"G": G, "P": P, "W": W, "M": M, "V": V, "seed": synth.matrix_seed(seed, s.index), "spec": s, **extra})
    return specs, items
