"""Helper of the guard-word test for the codec entry points (test-side only)."""
import numpy as np
import torch

from paper_2309_06973_b200 import binding as B


def run_guarded_codec(data: np.ndarray, Guarded):
    n = data.size
    nc = B.dnns_deflate_chunks(n)
    cap = (B.dnns_deflate_bound(n) + 3) // 4 * 4
    wsb = B.dnns_deflate_workspace_bytes(n)
    dev = "cuda"
    u8 = lambda k: torch.empty(k, dtype=torch.uint8, device=dev)
    g = {"src": Guarded(u8(n)), "stream": Guarded(u8(cap)), "ws": Guarded(u8(wsb)),
         "chunk_offset": Guarded(torch.empty(nc + 1, dtype=torch.int64, device=dev)),
         "sub_bits": Guarded(torch.empty(32 * nc, dtype=torch.int32, device=dev)),
         "dst": Guarded(u8(n)), "status": Guarded(torch.zeros(1, dtype=torch.int32, device=dev))}
    g["src"].view.copy_(torch.from_numpy(data))
    g["status"].view.zero_()
    st = torch.cuda.current_stream().cuda_stream
    B.dnns_deflate(g["src"].view.data_ptr(), n, g["stream"].view.data_ptr(), cap, g["chunk_offset"].view.data_ptr(),
                   g["sub_bits"].view.data_ptr(), g["ws"].view.data_ptr(), wsb, st)
    size = int(g["chunk_offset"].view[nc].item())
    B.dnns_inflate(g["stream"].view.data_ptr(), size, g["chunk_offset"].view.data_ptr(), g["sub_bits"].view.data_ptr(), n,
                   g["dst"].view.data_ptr(), g["status"].view.data_ptr(), st)
    torch.cuda.synchronize()
    assert int(g["status"].view.item()) == B.DNNS_OK
    assert np.array_equal(g["dst"].view.cpu().numpy(), data)
    for name, guard in g.items():
        assert guard.intact(), name
