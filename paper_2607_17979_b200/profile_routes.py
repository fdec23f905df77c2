"""Runs the persistent-state-pass route and the two-part route of the chunked prefill a few times on
the varlen benchmark batch (4 sequences {512,1024,2048,4096}, 32 v-heads), for a profiler's
launch list.  The two-part route is called with everything produced before the state pass
(split_permille=1000): a profiler that replays kernels one at a time cannot run a state pass that
waits for the launch behind it.

    python -m paper_2607_17979_b200.profile_routes
"""
import numpy as np
import torch

from paper_2607_17979_b200 import api, inputs as I


def main(reps=3):
    p = I.prefill_inputs([512, 1024, 2048, 4096], 16, 32, seed=1, init="zero")
    T, N, Hv = p["T"], p["N"], 32
    q, k, v = (torch.from_numpy(p[n].view(np.int16)).cuda().view(torch.bfloat16) for n in ("q", "k", "v"))
    g, beta, cu = (torch.from_numpy(p[n]).cuda() for n in ("g", "beta", "cu_seqlens"))
    ws = torch.zeros(api.gdn_prefill_workspace_bytes(T, N, 16, Hv), dtype=torch.uint8, device="cuda")
    final = torch.zeros((N, Hv, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.zeros((T, Hv, 128), dtype=torch.bfloat16, device="cuda")
    for _ in range(reps):
        api.gdn_prefill(q, k, v, g, beta, cu, None, final, None, o, p["scale"], ws, route="stream")
        api.gdn_prefill(q, k, v, g, beta, cu, None, final, None, o, p["scale"], ws, route="overlap",
                        split_permille=1000)
    torch.cuda.synchronize()
    print("ok")


if __name__ == "__main__":
    main()
