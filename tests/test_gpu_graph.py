"""A sequence (one quantiser launch, one persistent matmul launch, one finishing launch, chained by programmatic
dependent launches) can be captured into a CUDA graph once it has run once, and the replays give the eager bits."""
import pytest
import torch

from paper_2402_17764_b200 import binding as B
from paper_2402_17764_b200 import synthetic as S

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2402_17764_b200 import build
    build.build()
    B.load_library()
    assert torch.cuda.is_available()
    yield
    torch.cuda.synchronize()


@pytest.mark.parametrize("M", [1, 12, 40, 130])
def test_sequence_replays_in_a_cuda_graph(M):
    """1 and 12 tokens: the weight-streaming kernels; 40 tokens: the table-driven weight-stationary tensor-core kernel;
    130 tokens: the table-driven tensor-core GEMM."""
    shapes = S.decoder_layer_shapes(512, 1408, kv_dim=128)
    layers = []
    for mi, sh in enumerate(shapes * 2):
        W = S.latent_weights(sh.N, sh.K, 300 + mi, device="cuda")
        packed, gamma = B.quantize_weights(W)
        X = S.activations(M, sh.K, 300 + mi, device="cuda", outlier_frac=0.01, outlier_scale=10.0)
        layers.append((packed, gamma, X, torch.zeros((M, sh.N), dtype=torch.bfloat16, device="cuda"), sh.N))
    seq = B.Sequence(layers)
    seq.forward()                      # the first run sets the kernels' attributes: it stays outside the capture
    torch.cuda.synchronize()
    eager = [l[3].clone() for l in layers]
    assert B.poll_status(seq.workspace) == 0

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        seq.forward()                  # on the capture stream (the current stream inside the context)
    for _ in range(3):
        for l in layers:
            l[3].zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert B.poll_status(seq.workspace) == 0
        for l, want in zip(layers, eager):
            assert torch.equal(l[3].view(torch.int16), want.view(torch.int16))
    del graph
    seq.close()
