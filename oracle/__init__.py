"""CPU oracle for the MQGrad hot path: test infrastructure, never imported by the product."""
