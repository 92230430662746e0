"""The allocation-free attention entry point against the regular one.

Some users of the library run where cudaMalloc is not theirs to call: inside a process whose
device memory pool is owned by another allocator, or as a plug-in that only receives
pointers.  They cannot create an encoder (create allocates workspace), so
``wf_attention_f32_static`` keeps its index arrays in a fixed array inside the library.  This
file is collected last on purpose and checks two calls in a row, because the second call
finds the array holding the first call's contents."""
import numpy as np
import pytest

from oracle import wf_oracle as O
from paper_2412_11272_b200 import inputs as I
from tests._util import make_encoder

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_static_attention_matches_regular_entry_point_twice():
    from paper_2412_11272_b200.binding import WfError, wf_attention_f32_static
    d = 256
    shape = I.EncoderShape("s", 80, d, 0, 4, 256, "f32", n_ctx=2048)
    enc = make_encoder(shape, I.encoder_weights(0, shape), 16, 8192, 1000)
    rng = np.random.default_rng(21)
    for call, lens in enumerate(([700, 3, 129, 16, 17, 1500], [5, 2000, 31])):      # second call: shorter work list
        cu = np.concatenate([[0], np.cumsum(lens)])
        qkv_np = rng.normal(size=(cu[-1], 3 * d)).astype(np.float32)
        qkv = torch.as_tensor(qkv_np).cuda()
        want = enc.wf_attention(qkv, cu)
        got = torch.full((int(cu[-1]), d), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        wf_attention_f32_static(qkv, cu, d, got)
        torch.cuda.synchronize()
        if call == 1:       # the property in the entry point's name: the device's free memory has not moved
            assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.isfinite(got).all()
        assert float((got - want).abs().max()) <= 1e-5            # same kernel: the float32 parity bar is 1e-3
        i = 2                                                       # and one whole sequence against the oracle
        q, k, v = (qkv_np[cu[i]:cu[i + 1], j * d:(j + 1) * d].astype(np.float64) for j in range(3))
        ref = O.attention(q, k, v, 4)
        assert np.max(np.abs(got[cu[i]:cu[i + 1]].cpu().numpy() - ref)) <= 1e-4
    big = np.arange(0, 70000, 1000)
    with pytest.raises(WfError) as ei:
        wf_attention_f32_static(qkv, big, d, got)                  # 69,000 tokens > 65,536
    assert ei.value.status == "WF_ERR_CAPACITY"
    enc.close()
