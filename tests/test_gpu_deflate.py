"""GPU parity of dnns_deflate / dnns_inflate (Module 7 / Module 8): the stream and both index arrays
equal the oracle's byte for byte, zlib inflates the GPU's stream, and the GPU's inflation returns the
input."""
import zlib

import numpy as np
import pytest
import torch

from oracle import deflate_oracle as D
from oracle import oracle as O
from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import Deflater, DeviceModel, Session
from test_oracle_deflate import inputs, sparse_floats

pytestmark = pytest.mark.gpu


def roundtrip(data: np.ndarray, check_zlib=True):
    n = data.size
    src = torch.from_numpy(np.concatenate([data, np.zeros(16, np.uint8)])).cuda()
    df = Deflater(n)
    df.deflate(src, n)
    size = df.stream_bytes()
    got = df.stream[:size].cpu().numpy()
    want, want_off, want_sub = D.deflate(data)
    off, sub = df.index()
    assert size == want.size
    assert np.array_equal(off, want_off) and np.array_equal(sub, want_sub)
    assert np.array_equal(got, want)
    if check_zlib:
        assert zlib.decompress(got.tobytes(), wbits=-15) == data.tobytes()
    dst = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device="cuda")      # guard bytes behind the output
    df.inflate(dst, size)
    torch.cuda.synchronize()
    assert int(df.status.item()) == B.DNNS_OK
    back = dst.cpu().numpy()
    assert np.array_equal(back[:n], data) and np.all(back[n:] == 0xA5)
    return size


@pytest.mark.parametrize("name,data", list(inputs()), ids=[n for n, _ in inputs()])
def test_stream_and_index_equal_the_oracle(name, data):
    roundtrip(data)


def test_many_chunks_with_ragged_tail():
    rng = np.random.default_rng(21)
    parts = [sparse_floats(rng, 40 * D.CHUNK, 0.8), rng.integers(0, 256, 3 * D.CHUNK, dtype=np.uint8),
             np.zeros(5 * D.CHUNK + 1234, np.uint8), sparse_floats(rng, 11 * D.CHUNK + 77, 0.5, np.uint16)]
    roundtrip(np.concatenate(parts))


def test_rebuilt_variant_of_a_model():
    """A rebuilt ResNet-56 variant (what Module 7 receives from Module 4) deflates below its size and
    comes back bit for bit."""
    wl = W.resnet56()
    dm = DeviceModel(wl, B.DNNS_F32)
    ses = Session(dm, wl.scope, len(wl.ks), want_mask_bits=False, want_nz_map=False)
    ses.magnitude_threshold(wl.ks)
    ses.variant(len(wl.ks) - 1, fused=True)
    torch.cuda.synchronize()
    offs = ses.dst_offsets.cpu().numpy().view(np.uint64)
    used = int(offs[-1]) + 256
    data = ses.compact_arena[:used].cpu().numpy().copy()
    size = roundtrip(data)
    assert size < 0.6 * used
    ses.close()


def test_damaged_stream_sets_the_status_word():
    data = np.zeros(3 * D.CHUNK, np.uint8)
    df = Deflater(data.size)
    df.deflate(torch.from_numpy(data).cuda(), data.size)
    size = df.stream_bytes()
    df.stream[0] = 0x04                      # BTYPE 10 (dynamic codes): never written by dnns_deflate
    dst = torch.zeros(data.size, dtype=torch.uint8, device="cuda")
    df.inflate(dst, size)
    torch.cuda.synchronize()
    assert int(df.status.item()) == B.DNNS_ERR_UNSUPPORTED


def test_host_side_argument_errors():
    df = Deflater(1000)
    src = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.DnnsError) as e:
        B.dnns_deflate(src.data_ptr(), 1000, df.stream.data_ptr(), 100, df.chunk_offset.data_ptr(),
                       df.sub_bits.data_ptr(), df.ws.data_ptr(), df.ws_bytes)
    assert e.value.status == B.DNNS_ERR_WORKSPACE
    with pytest.raises(B.DnnsError) as e:
        B.dnns_deflate(src.data_ptr() + 4, 1000, df.stream.data_ptr(), df.capacity, df.chunk_offset.data_ptr(),
                       df.sub_bits.data_ptr(), df.ws.data_ptr(), df.ws_bytes)
    assert e.value.status == B.DNNS_ERR_INVALID_ARG
